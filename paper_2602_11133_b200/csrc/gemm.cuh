// Persistent, warp-specialised bf16 GEMM for sm_100a:  D[M, N] = A[M, K] . W[N, K]^T, fp32 accumulate.
//
//   warp 0 (one lane)  TMA producer: 128 x 64 tile of A and BN x 64 tile of W per pipeline stage
//   warp 1 (one lane)  tcgen05.mma issuer (UMMA 128 x BN x 16), accumulators in tensor memory,
//                      two accumulator buffers so the epilogue of tile t overlaps the MMAs of tile t+1
//   warps 2..5         epilogue: each thread owns one accumulator row (TMEM lane), reads it 32 columns
//                      at a time and applies one of three epilogues:
//        EPI_STORE   bf16(acc [+ residual])                                  -> C[M, N]
//        EPI_SWIGLU  bf16(silu(gate) * up), gate/up from the two halves of W -> C[M, N/2]
//        EPI_STATS   online (max, argmax, runner-up, sum-exp) per row over a range of vocabulary tiles
//                    (EPI_STATS_DRAW: plus one Gumbel-max draw per row);
//                    the logits are never written (LM head of the denoising step)
//        EPI_QKV     QKV projection: bf16(acc), then rotary embedding on the Q and K heads (rotate-half,
//                    table lookup by canvas position) written to C, and the V heads written transposed
//                    (keys contiguous) for the attention kernel's P.V product
//        EPI_PARTIAL fp32 partial sums of one K range (split-K for projections with too few output
//                    tiles to fill the SMs); splitk_reduce_kernel adds the ranges and the residual
#pragma once
#include "pdl.cuh"
#include "ptx.cuh"

namespace jot {

enum { EPI_STORE = 0, EPI_SWIGLU = 1, EPI_STATS = 2, EPI_PARTIAL = 3, EPI_QKV = 4, EPI_STATS_DRAW = 5 };
// EPI_STATS_DRAW is EPI_STATS plus the Gumbel-max draw of sampling-based finalisation: an instance of its own, so
// that the argmax-only head does not carry the draw's registers.
__host__ __device__ constexpr bool is_stats(int epi) { return epi == EPI_STATS || epi == EPI_STATS_DRAW; }

// Pipeline depth (shared-memory stages of one A tile + one W tile); both fill ~192 KB.
#ifndef JOT_GEMM_STAGES_256
#define JOT_GEMM_STAGES_256 4
#endif
#ifndef JOT_GEMM_STAGES_128
#define JOT_GEMM_STAGES_128 6
#endif

constexpr int kBM = 128;          // rows per tile = TMEM lanes
constexpr int kBK = 64;           // bf16 elements per 128-byte swizzled smem row
constexpr int kGemmThreads = 192;

struct GemmParams {
    int M, N, K;                  // N = rows of W (for EPI_SWIGLU: 2 * d_ff)
    __nv_bfloat16* C;             // EPI_STORE / EPI_SWIGLU output
    const __nv_bfloat16* residual;  // EPI_STORE, nullable, same shape as C
    int ldc;                      // row stride of C and residual, elements
    int32_t* status;              // set non-zero when a bounded wait expired (nullable)
    int split_k;                  // EPI_PARTIAL: number of K ranges (>= 1); otherwise ignored
    float* partial;               // EPI_PARTIAL: [split_k][M][N] fp32
    // EPI_QKV only: C = qkv [B * L, (nq + 2 nkv) * hd].  The launch covers rows_per_seq consecutive canvas
    // positions of every sequence, starting at pos0: input row r is (sequence, position) =
    // (r / rows_per_seq, pos0 + r % rows_per_seq) and lands in row sequence * L + position of C and of V^T.
    // The whole canvas is rows_per_seq = L, pos0 = 0; a block-wise KV cache recomputes one block's rows.
    __nv_bfloat16* vt;            // [B * nkv * hd, Lp] V transposed
    const float2* rope_cs;        // [max_seq, hd / 2] (cos, sin)
    int L, Lp, nq, nkv, hd;
    int rows_per_seq, pos0;
    // EPI_STATS only
    const int32_t* d_R;           // number of active rows (device)
    const int32_t* rows;          // [R] flat canvas index b*L+i of each active row
    const int32_t* bump_id;       // nullable, indexed by flat canvas index
    const float* bump_val;
    int mask_col;                 // column to exclude, or -1
    int col_lo, col_hi;           // vocabulary slice [col_lo, col_hi) the statistics cover (col_hi = 0: all N columns)
    float4* partials;             // [chunks][R_pad] (m1, bitcast i1, m2, S)
    // sampling-based finalisation (inv_temperature > 0): each row also draws a token from softmax(l / T)
    float inv_temperature;
    unsigned long long sample_seed;
    const int32_t* d_seq_steps;   // generate loop: steps_used of sequence b at d_seq_steps[4 * b] (nullable: then
    int step_value;               // step_value); b = flat canvas index / L
    float2* partials2;            // [chunks][R_pad] (best perturbed score, bitcast token)
    int R_pad;                    // row capacity of one chunk of partials (multiple of 128)
    // slab kernel only (gemm_slab.cuh): first pair-slab of the launch and pairs per cluster (K ranges)
    int slab0, slab_split;
};

template <int BN>
struct GemmSmem {
    static constexpr int A_BYTES = kBM * kBK * 2;
    static constexpr int B_BYTES = BN * kBK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = (BN == 256) ? JOT_GEMM_STAGES_256 : JOT_GEMM_STAGES_128;
    static constexpr int STAGING_BYTES = 4 * 32 * 36 * 4;          // per epilogue warp 32 x 36 floats (EPI_PARTIAL)
    static constexpr int DYN_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + 1024;   // + slack to align to 1024
};

// How the stats kernel splits the vocabulary: row blocks run side by side over the same vocabulary
// range so that a tile of W fetched from HBM by one CTA is found in L2 by the others.
__host__ __device__ inline void stats_partition(int R, int grid, int n_vt, int* n_rb, int* n_ch) {
    int rb = (R + kBM - 1) / kBM;
    int ch = rb > 0 ? grid / rb : 0;
    if (ch > n_vt) ch = n_vt;
    *n_rb = rb;
    *n_ch = ch;
}

// Running LM-head statistics of one output row (EPI_STATS), carried across the vocabulary tiles a CTA visits.
struct StatsRow {
    float m1 = -INFINITY, m2 = -INFINITY, S = 0.f;
    int i1 = 0x7fffffff;
    int bump_col = -1;
    float bump_v = 0.f;
    float best = -INFINITY;       // Gumbel-max draw: largest perturbed score so far and its token
    int best_i = 0x7fffffff;
    unsigned long long key = 0;   // start state of this row's random stream
};

// splitmix64 output function (Steele, Lea, Flood 2014); output number n of the stream with start state k is
// mix64(k + n * 0x9E3779B97F4A7C15).
__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// Per-row set-up of the LM-head epilogue: planted bump and, when sampling, the key of the row's stream
// (seed, step and flat canvas position mixed together).
__device__ __forceinline__ void stats_row_init(const GemmParams& p, int row, StatsRow& st) {
    if (row >= *p.d_R) return;
    const int flat = p.rows[row];
    if (p.bump_id != nullptr) {
        st.bump_col = p.bump_id[flat];
        st.bump_v = p.bump_val[flat];
    }
    if (p.inv_temperature > 0.f) {
        const unsigned long long step =
            (unsigned long long)(p.d_seq_steps ? p.d_seq_steps[4 * (flat / p.L)] : p.step_value);
        st.key = mix64(p.sample_seed ^ (step << 40) ^ (unsigned long long)flat);
    }
}

// Epilogue of one 128 x BN accumulator tile: the calling thread owns output row `row` (TMEM lane) and reads
// it 32 columns at a time from tensor memory at `t_acc`.  Shared by the one-CTA and the CTA-pair kernels.
template <int BN, int EPI>
__device__ __forceinline__ void epilogue_tile(const GemmParams& p, uint32_t t_acc, int row, int n_blk, int ks,
                                              int n_out, StatsRow& st, float* stg = nullptr) {
    constexpr float L2E = 1.4426950408889634f;
    (void)L2E; (void)ks; (void)n_out; (void)st;
    if (EPI == EPI_STORE) {
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            float v[32];
            tmem_ld32(t_acc + c * 32, v);
            tmem_ld_wait();
            const int col0 = n_blk * BN + c * 32;
            if (row < p.M) {
                __nv_bfloat16* dst = p.C + (size_t)row * p.ldc + col0;
                const __nv_bfloat16* res = p.residual ? p.residual + (size_t)row * p.ldc + col0 : nullptr;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    if (col0 + g * 8 < p.N) {         // N is a multiple of 8
                        float x[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) x[j] = v[g * 8 + j];
                        if (res) {
                            uint4 rv = *reinterpret_cast<const uint4*>(res + g * 8);
                            const __nv_bfloat162* r2 = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                float2 f = __bfloat1622float2(r2[j]);
                                x[2 * j] += f.x;
                                x[2 * j + 1] += f.y;
                            }
                        }
                        uint4 ov;
                        __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
                        for (int j = 0; j < 4; ++j) o2[j] = __floats2bfloat162_rn(x[2 * j], x[2 * j + 1]);
                        *reinterpret_cast<uint4*>(dst + g * 8) = ov;
                    }
                }
            }
        }
    } else if (EPI == EPI_QKV) {
        const int hd = p.hd, half = hd >> 1;
        const int seq = row / p.rows_per_seq, pos = p.pos0 + (row - seq * p.rows_per_seq);
        const size_t dst_row = (size_t)seq * p.L + pos;
#pragma unroll 1
        for (int hh = 0; hh < BN / hd; ++hh) {
            const int col_base = n_blk * BN + hh * hd;
            if (col_base >= p.N) break;
            const int head = col_base / hd;
            if (head < p.nq + p.nkv) {
                // rotate pairs (j, j + hd/2): 32 pairs at a time
#pragma unroll 1
                for (int q = 0; q < half / 32; ++q) {
                    float lo[32], hi[32];
                    tmem_ld32(t_acc + hh * hd + q * 32, lo);
                    tmem_ld32(t_acc + hh * hd + half + q * 32, hi);
                    tmem_ld_wait();
                    if (row < p.M) {
                        const float4* cs4 = reinterpret_cast<const float4*>(p.rope_cs + (size_t)pos * half + q * 32);
                        __nv_bfloat16* dlo = p.C + dst_row * p.ldc + col_base + q * 32;
                        __nv_bfloat16* dhi = dlo + half;
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            uint4 olo, ohi;
                            __nv_bfloat162* l2 = reinterpret_cast<__nv_bfloat162*>(&olo);
                            __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&ohi);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const int e = g * 8 + 2 * j;
                                const float4 k = cs4[e >> 1];      // (cos, sin) of pairs e and e + 1
                                // the projection's output is bf16; the rotation acts on the rounded values
                                const float2 x0 = __bfloat1622float2(__floats2bfloat162_rn(lo[e], lo[e + 1]));
                                const float2 x1 = __bfloat1622float2(__floats2bfloat162_rn(hi[e], hi[e + 1]));
                                l2[j] = __floats2bfloat162_rn(x0.x * k.x - x1.x * k.y, x0.y * k.z - x1.y * k.w);
                                h2[j] = __floats2bfloat162_rn(x1.x * k.x + x0.x * k.y, x1.y * k.z + x0.y * k.w);
                            }
                            *reinterpret_cast<uint4*>(dlo + g * 8) = olo;
                            *reinterpret_cast<uint4*>(dhi + g * 8) = ohi;
                        }
                    }
                }
            } else {
                // V head: lane = position, so for a fixed d a warp writes 32 consecutive keys
                const int kvh = head - p.nq - p.nkv;
#pragma unroll 1
                for (int c = 0; c < hd / 32; ++c) {
                    float v[32];
                    tmem_ld32(t_acc + hh * hd + c * 32, v);
                    tmem_ld_wait();
                    if (row < p.M) {
                        __nv_bfloat16* dst = p.vt + ((size_t)(seq * p.nkv + kvh) * hd + c * 32) * p.Lp + pos;
#pragma unroll
                        for (int j = 0; j < 32; ++j) dst[(size_t)j * p.Lp] = __float2bfloat16_rn(v[j]);
                    }
                }
            }
        }
    } else if (EPI == EPI_PARTIAL) {
        // A thread owns a row, so its 32 columns are 128 contiguous bytes, but a warp's rows lie N * 4 bytes
        // apart.  The warp turns its 32 x 32 block around through `stg` (rows padded to 36 floats: no bank
        // conflicts either way) so that every store instruction covers four whole 128-byte lines.
        const int lane = threadIdx.x & 31;
        const int row0 = row - lane;                          // first row of this warp's block
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            float v[32];
            tmem_ld32(t_acc + c * 32, v);
            tmem_ld_wait();
            const int col0 = n_blk * BN + c * 32;
#pragma unroll
            for (int g = 0; g < 8; ++g)
                *reinterpret_cast<float4*>(stg + lane * 36 + g * 4) = make_float4(v[g * 4], v[g * 4 + 1], v[g * 4 + 2], v[g * 4 + 3]);
            __syncwarp();
            const int cg = lane & 7;                          // four columns of the row
            if (col0 + cg * 4 < p.N) {                        // N is a multiple of 8
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const int r = it * 4 + (lane >> 3);
                    if (row0 + r < p.M)
                        *reinterpret_cast<float4*>(p.partial + ((size_t)ks * p.M + row0 + r) * p.N + col0 + cg * 4) =
                            *reinterpret_cast<const float4*>(stg + r * 36 + cg * 4);
                }
            }
            __syncwarp();
        }
    } else if (EPI == EPI_SWIGLU) {
#pragma unroll 1
        for (int c = 0; c < BN / 64; ++c) {
            float g[32], u[32];
            tmem_ld32(t_acc + c * 32, g);
            tmem_ld32(t_acc + BN / 2 + c * 32, u);
            tmem_ld_wait();
            const int col0 = n_blk * (BN / 2) + c * 32;
            if (row < p.M) {
                __nv_bfloat16* dst = p.C + (size_t)row * p.ldc + col0;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (col0 + q * 8 < n_out) {
                        uint4 ov;
                        __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float g0 = g[q * 8 + 2 * j], g1 = g[q * 8 + 2 * j + 1];
                            float a0 = g0 / (1.f + __expf(-g0)) * u[q * 8 + 2 * j];
                            float a1 = g1 / (1.f + __expf(-g1)) * u[q * 8 + 2 * j + 1];
                            o2[j] = __floats2bfloat162_rn(a0, a1);
                        }
                        *reinterpret_cast<uint4*>(dst + q * 8) = ov;
                    }
                }
            }
        }
    } else {
        // ---- EPI_STATS: fold this tile's logits into (st.m1, st.i1, st.m2, st.S) ----
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            float v[32];
            tmem_ld32(t_acc + c * 32, v);
            tmem_ld_wait();
            const int col0 = n_blk * BN + c * 32;
            const int hi_col = p.col_hi > 0 ? p.col_hi : p.N;      // the statistics cover columns [col_lo, hi_col)
            if (col0 >= hi_col) break;                    // whole chunk past the slice
            if (col0 + 32 <= p.col_lo) continue;          // whole chunk before it
            unsigned rel_b = (unsigned)(st.bump_col - col0);
            if (rel_b < 32u) {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] += (j == (int)rel_b) ? st.bump_v : 0.f;
            }
            unsigned rel_m = (unsigned)(p.mask_col - col0);
            if (p.mask_col >= 0 && rel_m < 32u) {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = (j == (int)rel_m) ? -INFINITY : v[j];
            }
            if (col0 + 32 > hi_col || col0 < p.col_lo) {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = (col0 + j < hi_col && col0 + j >= p.col_lo) ? v[j] : -INFINITY;
            }
            if (EPI == EPI_STATS_DRAW) {
                // Gumbel-max: argmax_v (l_v / T - ln(-ln u_v)), u_v from 23 bits of the row's counter stream
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const unsigned long long z = mix64(st.key + (unsigned long long)(col0 + j + 1) * 0x9E3779B97F4A7C15ull);
                    const float u = ((float)(unsigned)(z >> 41) + 0.5f) * (1.f / 8388608.f);
                    const float score = fmaf(v[j], p.inv_temperature, -logf(-logf(u)));
                    if (score > st.best) {               // strict: the lowest token id wins ties
                        st.best = score;
                        st.best_i = col0 + j;
                    }
                }
            }
            float cm = v[0];
#pragma unroll
            for (int j = 1; j < 32; ++j) cm = fmaxf(cm, v[j]);
            const float old_m = st.m1;
            if (cm > st.m2) {                                // only then can the top two change
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float x = v[j];
                    st.m2 = fmaxf(st.m2, fminf(x, st.m1));         // runner-up as an order statistic
                    st.i1 = (x > st.m1) ? col0 + j : st.i1;        // strict: the lowest index wins ties
                    st.m1 = fmaxf(st.m1, x);
                }
            }
            if (st.m1 == -INFINITY) continue;                // nothing but excluded columns so far: no sum yet
            // st.S = sum exp(l - st.m1): rescale what was summed against the old maximum
            const float nm = st.m1 * L2E;
            float acc_s = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j) acc_s += ex2_approx(fmaf(v[j], L2E, -nm));
            st.S = st.S * ex2_approx(old_m * L2E - nm) + acc_s;
        }
    }
}

template <int BN, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const GemmParams p, const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB) {
    using SM = GemmSmem<BN>;
    constexpr int STAGES = SM::STAGES;
    constexpr uint32_t TMEM_COLS = 2 * BN;                 // 256 or 512, a power of two
    constexpr uint32_t IDESC = umma_idesc_bf16(kBM, BN);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (p.K + kBK - 1) / kBK;

    // ---- setup ----
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&acc_full[a], 1);
            mbar_init(&acc_empty[a], 4);
        }
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(&tmem_base_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    // everything above is on-chip; from here on global memory written by earlier kernels is read.  The LM-head
    // schedule depends on a device word the preceding kernel wrote, so that kernel waits here; the others let
    // every role wait for itself, and the producer requests its first W tiles BEFORE it waits (the weights are
    // nobody's output): the pipeline fill overlaps the predecessor's tail.
    grid_launch_dependents();
    if (is_stats(EPI)) grid_dependency_wait();


    // ---- tile schedule (identical in every role) ----
    int m_blk0 = 0, n_first = 0, n_count = 0;      // EPI_STATS: one row block, a range of vocabulary tiles
    int num_m = (p.M + kBM - 1) / kBM;
    constexpr int BN_OUT = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
    const int n_out = (EPI == EPI_SWIGLU) ? p.N / 2 : p.N;
    const int num_n = (n_out + BN_OUT - 1) / BN_OUT;
    const int split = (EPI == EPI_PARTIAL) ? p.split_k : 1;
    int total_tiles = num_m * num_n * split;
    int chunk = 0;
    // EPI_STATS: only the tiles that touch the vocabulary slice are visited
    const int stats_hi = (is_stats(EPI) && p.col_hi > 0) ? p.col_hi : p.N;
    const int tile_lo = (is_stats(EPI)) ? p.col_lo / BN : 0;
    const int num_nt = (is_stats(EPI)) ? (stats_hi + BN - 1) / BN - tile_lo : num_n;
    if (is_stats(EPI)) {
        int R = *p.d_R, n_rb, n_ch;
        stats_partition(R, gridDim.x, num_nt, &n_rb, &n_ch);
        chunk = n_rb > 0 ? blockIdx.x / n_rb : 0;
        if (n_rb == 0 || chunk >= n_ch) {
            n_count = 0;
        } else {
            m_blk0 = blockIdx.x % n_rb;
            n_first = (int)((long long)chunk * num_nt / n_ch);
            n_count = (int)((long long)(chunk + 1) * num_nt / n_ch) - n_first;
            n_first += tile_lo;
        }
        total_tiles = n_count;
    }
    int kb0 = 0, kb1 = num_kb, ks = 0;            // K-block range of the current work item
    auto tile_at = [&](int it, int& m_blk, int& n_blk) -> bool {
        if (is_stats(EPI)) {
            if (it >= total_tiles) return false;
            m_blk = m_blk0;
            n_blk = n_first + it;
            return true;
        }
        int t = blockIdx.x + it * gridDim.x;
        if (t >= total_tiles) return false;
        if (EPI == EPI_PARTIAL) {
            ks = t % split;
            t /= split;
            kb0 = (int)((long long)ks * num_kb / split);
            kb1 = (int)((long long)(ks + 1) * num_kb / split);
        }
        m_blk = t % num_m;                        // row blocks fastest: neighbours share the W tile
        n_blk = t / num_m;
        return true;
    };

    if (warp == 0) {
        // ================= TMA producer (the whole warp runs the loop, one lane issues) =================
        const bool elected = elect_one();
        int stage = 0;
        uint32_t phase = 0;
        int m_blk, n_blk;
        bool ok = true;
        auto load_w = [&](int st, int kb, int nb) {
            uint8_t* sB = smem + st * SM::STAGE_BYTES + SM::A_BYTES;
            mbar_arrive_expect_tx(&full_bar[st], SM::STAGE_BYTES);
            if (EPI == EPI_SWIGLU) {
                // gate rows, then the matching up rows: two boxes of BN/2 rows each
                tma_load_2d(sB, &tmB, &full_bar[st], kb * kBK, nb * (BN / 2));
                tma_load_2d(sB + SM::B_BYTES / 2, &tmB, &full_bar[st], kb * kBK, p.N / 2 + nb * (BN / 2));
            } else {
                tma_load_2d(sB, &tmB, &full_bar[st], kb * kBK, nb * BN);
            }
        };
        // the first tile's first W tiles go out before the wait on the preceding kernel, its A tiles after
        int n_pre = 0;
        if (!is_stats(EPI)) {
            if (tile_at(0, m_blk, n_blk)) {
                n_pre = min(STAGES, kb1 - kb0);
                if (elected)
                    for (int i = 0; i < n_pre; ++i) load_w(i, kb0 + i, n_blk);
            }
            __syncwarp();
            grid_dependency_wait();
            if (elected)
                for (int i = 0; i < n_pre; ++i)
                    tma_load_2d(smem + i * SM::STAGE_BYTES, &tmA, &full_bar[i], (kb0 + i) * kBK, m_blk * kBM);
            __syncwarp();
        }
        for (int it = 0; ok && tile_at(it, m_blk, n_blk); ++it) {
            for (int kb = kb0; kb < kb1; ++kb) {
                if (it == 0 && kb - kb0 < n_pre) {            // already requested above
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    continue;
                }
                if (!mbar_wait(&empty_bar[stage], phase ^ 1, abortp)) { ok = false; break; }
                if (elected) {
                    load_w(stage, kb, n_blk);
                    tma_load_2d(smem + stage * SM::STAGE_BYTES, &tmA, &full_bar[stage], kb * kBK, m_blk * kBM);
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer (the whole warp runs the loop, one lane issues) =================
        // The operand descriptors of a stage differ from stage 0's only in the 16-byte-granular address field
        // and are advanced by additions (the field never carries: shared-memory addresses stay below 256 KB).
        const bool elected = elect_one();
        const uint64_t ad0 = umma_desc_k128(smem_u32(smem));
        const uint64_t bd0 = ad0 + (SM::A_BYTES >> 4);
        constexpr uint32_t STAGE_UNITS = SM::STAGE_BYTES >> 4;
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        uint64_t ad = ad0, bd = bd0;
        int m_blk, n_blk;
        bool ok = true;
        for (int it = 0; ok && tile_at(it, m_blk, n_blk); ++it) {
            if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1, abortp)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * BN;
            uint32_t accum = 0;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!mbar_wait(&full_bar[stage], phase, abortp)) { ok = false; break; }
                tc_fence_after();
                if (elected) {
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) umma_bf16(d_tmem, ad + 2 * k, bd + 2 * k, IDESC, accum | k);
                    umma_commit(&empty_bar[stage]);       // smem stage reusable once these MMAs retire
                }
                __syncwarp();
                accum = 1;
                ad += STAGE_UNITS;
                bd += STAGE_UNITS;
                if (++stage == STAGES) { stage = 0; phase ^= 1; ad = ad0; bd = bd0; }
            }
            if (!ok) break;
            if (elected) umma_commit(&acc_full[acc]);     // accumulator complete
            __syncwarp();
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        __syncwarp();
    } else {
        // ================= epilogue (warps 2..5) =================
        if (!is_stats(EPI)) grid_dependency_wait();     // residual, rotary table: written or read after earlier kernels
        const int quad = warp & 3;                        // TMEM lanes [32*quad, 32*quad+32)
        const int row_in_tile = quad * 32 + lane;
        const uint32_t lane_base = tmem_base + (uint32_t(quad * 32) << 16);
        int acc = 0;
        uint32_t acc_phase = 0;
        int m_blk, n_blk;
        StatsRow st;
        if (is_stats(EPI) && total_tiles > 0) stats_row_init(p, m_blk0 * kBM + row_in_tile, st);
        bool ok = true;
        for (int it = 0; ok && tile_at(it, m_blk, n_blk); ++it) {
            if (!mbar_wait(&acc_full[acc], acc_phase, abortp)) { ok = false; break; }
            tc_fence_after();
            epilogue_tile<BN, EPI>(p, lane_base + acc * BN, m_blk * kBM + row_in_tile, n_blk, ks, n_out, st,
                                   reinterpret_cast<float*>(smem + STAGES * SM::STAGE_BYTES) + quad * (32 * 36));
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[acc]);
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        if (is_stats(EPI) && ok && total_tiles > 0) {
            const size_t slot = (size_t)chunk * p.R_pad + m_blk0 * kBM + row_in_tile;
            p.partials[slot] = make_float4(st.m1, __int_as_float(st.i1), st.m2, st.S);
            if (EPI == EPI_STATS_DRAW) p.partials2[slot] = make_float2(st.best, __int_as_float(st.best_i));
        }
    }

    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
    if (threadIdx.x == 0 && abort_flag && p.status) atomicExch(p.status, 1);
}

// C = bf16( sum over K ranges of partial + residual ).  8 outputs per thread.
__global__ void splitk_reduce_kernel(const float* __restrict__ partial, int split, const __nv_bfloat16* residual,
                                     __nv_bfloat16* C, int M, int N) {
    grid_launch_dependents();
    grid_dependency_wait();
    const size_t i8 = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 8;
    const size_t total = (size_t)M * N;
    if (i8 >= total) return;
    float x[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) x[j] = 0.f;
    for (int s = 0; s < split; ++s) {
        const float4 a = *reinterpret_cast<const float4*>(partial + s * total + i8);
        const float4 b = *reinterpret_cast<const float4*>(partial + s * total + i8 + 4);
        x[0] += a.x; x[1] += a.y; x[2] += a.z; x[3] += a.w;
        x[4] += b.x; x[5] += b.y; x[6] += b.z; x[7] += b.w;
    }
    if (residual) {
        const uint4 rv = *reinterpret_cast<const uint4*>(residual + i8);
        const __nv_bfloat162* r2 = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __bfloat1622float2(r2[j]);
            x[2 * j] += f.x;
            x[2 * j + 1] += f.y;
        }
    }
    uint4 ov;
    __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
    for (int j = 0; j < 4; ++j) o2[j] = __floats2bfloat162_rn(x[2 * j], x[2 * j + 1]);
    *reinterpret_cast<uint4*>(C + i8) = ov;
}

}  // namespace jot
