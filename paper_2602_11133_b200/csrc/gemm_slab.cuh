// Projection kernel for small canvases (at most 512 rows): the weight rows are the MMA's M side.
//
//   D^T[feature, token] = W[feature, :] . X[token, :]^T      (fp32 in tensor memory, bf16 operands, both K-major)
//
// With few tokens the projection is a stream of W against a small X.  A 128 x 256 token-major tile takes in
// 48 KB of operands per 4.2 MFLOP, which the SM's operand ingest (not HBM, not the tensor pipe) limits.  Here
// a CTA pair (tcgen05 cta_group::2, UMMA M = 256) owns a slab of 256 weight rows, 128 per CTA, and ALL tokens
// are the N side: one or two accumulators of up to 256 token columns each.  Per CTA and k-block of 64 that
// is 16 KB of W plus half of the token tile (the pair splits the N operand), e.g. 16 + 24 KB for 6.3 MFLOP at
// 384 tokens: every W byte enters exactly one SM and the token tile is the only operand fetched repeatedly.
//
//   warp 0 (one lane)  TMA producer (both CTAs of the pair): W box, then this CTA's half of every token box
//   warp 1 (one lane)  MMA issuer (even CTA of the pair): per k-step one UMMA per accumulator
//   warps 2..9         epilogue, two warps per TMEM lane quadrant (a lane is an output FEATURE)
//
// Split-K inside a cluster: a cluster is S pairs (S = 1..4) that cut K into S ranges.  After the main loop
// the pairs exchange partial sums through distributed shared memory as a reduce-scatter over tokens: pair q
// becomes the owner of the q-th range of token chunks, receives the other pairs' partial sums for it
// (plain st.shared::cluster stores, no multicast), adds them in a fixed order and runs the epilogue for its
// range.  No scratch in global memory, no second kernel, the same bits on every run.
//
// Epilogue: a thread holds one feature and 32 consecutive tokens, the outputs are token-major.  Each group
// of four warps (128 features) turns its 32-token chunk around through a 16 KB fp32 buffer in shared memory
// (the pipeline's stages, free by then) and leaves with 16-byte stores:
//     SLAB_STORE   bf16(acc [+ residual])
//     SLAB_SWIGLU  a CTA's 128 rows are 64 gate rows and the matching 64 up rows: bf16(silu(g) * u)
//     SLAB_QKV     bf16(acc), rotary embedding on Q and K heads (the partner feature sits 64 lanes away, the
//                  buffer brings them together), V heads written transposed straight from the registers
//                  (a thread's 32 tokens are 64 contiguous bytes of V^T)
#pragma once
#include "gemm.cuh"

namespace jot {

constexpr int kSlabThreads = 320;
constexpr int kSlabMaxTokens = 512;        // two accumulators of 256 fp32 columns fill tensor memory
#ifndef JOT_SLAB_PREFER_TOKENS
#define JOT_SLAB_PREFER_TOKENS 256
#endif
constexpr int kSlabPreferTokens = JOT_SLAB_PREFER_TOKENS;   // measured: up to here this kernel beats the token-major tiles
#ifndef JOT_SLAB_GATEUP_TOKENS
#define JOT_SLAB_GATEUP_TOKENS JOT_SLAB_PREFER_TOKENS
#endif
constexpr int kSlabGateUpTokens = JOT_SLAB_GATEUP_TOKENS;   // the same switch for the gate/up projection alone
constexpr int kSlabMaxSmem = 226 * 1024;   // dynamic part; the static barriers take the rest of the 227 KB
enum { SLAB_STORE = 0, SLAB_SWIGLU = 1, SLAB_QKV = 2 };

// How a canvas of M rows maps onto accumulators, and what a launch needs in shared memory.  The tensor pipe
// spends as long on a UMMA of 192 columns as on one of 256 (measured), so the first accumulator always
// takes 256 tokens when there are more than that and the second one the rest.
struct SlabGeom {
    int n_acc;          // accumulators (UMMAs per k-step)
    int n0, n1;         // token columns of the two accumulators: multiples of 32, at most 256 (n1 = 0: one only)
    int n_chunks;       // 32-token chunks over all accumulators
    int stage_bytes;    // W tile + this CTA's half of every token tile
    int stages;
    int cpo;            // chunks per owner after the reduce-scatter (all of them when split == 1)
    int recv_bytes;     // partial sums received from the other split ranks
    int smem_bytes;     // dynamic shared memory of the launch
};

__host__ __device__ inline SlabGeom slab_geom(int M, int split) {
    SlabGeom g;
    g.n_acc = M > 256 ? 2 : 1;
    g.n0 = g.n_acc == 2 ? 256 : (M + 31) / 32 * 32;
    if (g.n0 < 32) g.n0 = 32;
    g.n1 = g.n_acc == 2 ? (M - 256 + 31) / 32 * 32 : 0;
    g.n_chunks = (g.n0 + g.n1) / 32;
    g.stage_bytes = 128 * 128 + ((g.n0 + g.n1) / 2) * 128;
    g.cpo = (g.n_chunks + split - 1) / split;
    g.recv_bytes = (split - 1) * g.cpo * 32 * 512;                // [source][token][128 features] fp32
    const int epi_bytes = g.recv_bytes + 4 * 32 * 512;            // + two fp32 chunk buffers per warp group
    int stages = (kSlabMaxSmem - 2048) / g.stage_bytes;
    if (stages > 12) stages = 12;      // few tokens: small stages, and the weight stream wants many bytes in flight
    g.stages = stages;
    const int pipe = stages * g.stage_bytes;
    g.smem_bytes = (pipe > epi_bytes ? pipe : epi_bytes) + 1024;
    return g;
}

#ifdef JOT_SLAB_TRACE
// Timestamps (nanoseconds of %globaltimer) of the latest launch with epilogue JOT_SLAB_TRACE, 16 words per CTA;
// only in instrumented builds (-DJOT_SLAB_TRACE=<epilogue>).
__device__ unsigned long long g_slab_trace[1024 * 16];
#define SLAB_TRACE(slot) do { if (EPI == JOT_SLAB_TRACE && blockIdx.x < 1024) g_slab_trace[blockIdx.x * 16 + (slot)] = global_ns(); } while (0)
#define SLAB_TRACE_VAL(slot, v) do { if (EPI == JOT_SLAB_TRACE && blockIdx.x < 1024) g_slab_trace[blockIdx.x * 16 + (slot)] = (v); } while (0)
#else
#define SLAB_TRACE(slot) do { } while (0)
#define SLAB_TRACE_VAL(slot, v) do { } while (0)
#endif

template <int EPI>
__global__ void __launch_bounds__(kSlabThreads, 1)
gemm_slab_kernel(const GemmParams p, const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                 const __grid_constant__ CUtensorMap tmX1) {
    constexpr int MAX_STAGES = 12;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t full_bar[MAX_STAGES], empty_bar[MAX_STAGES], acc_full;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = p.slab_split;                             // pairs per cluster
    const uint32_t rank = cluster_ctarank();                    // 0 .. 2 * split - 1
    const int pr = (int)(rank & 1u), ks = (int)(rank >> 1);     // rank inside the pair, K range of the pair
    const uint32_t leader_rank = rank & ~1u;
    const bool leader = pr == 0;
    const int slab = p.slab0 + (int)(blockIdx.x / (2 * split)); // pair-slab: 256 weight rows (128 outputs for SwiGLU)
    const SlabGeom g = slab_geom(p.M, split);
    const int stages = g.stages;
    const int h0 = g.n0 / 2, h1 = g.n1 / 2;                      // token rows this CTA loads per accumulator
    const int num_kb = (p.K + kBK - 1) / kBK;
    const int kb0 = (int)((long long)ks * num_kb / split), kb1 = (int)((long long)(ks + 1) * num_kb / split);
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < g.n0 + g.n1) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&acc_full, 1);
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmX);
        tma_prefetch_desc(&tmX1);
    }
    if (warp == 1) {
        tmem_alloc_pair(&tmem_base_slot, tmem_cols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    cluster_sync_all();                       // every CTA's barriers exist before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    if (threadIdx.x == 0) SLAB_TRACE(0);
    grid_launch_dependents();
    // Every role waits for the preceding kernel (grid_dependency_wait) before it touches what that kernel wrote:
    // the activations, the residual.  The weights are nobody's output, so the producer requests the first W
    // tiles BEFORE that wait and the pipeline's fill latency overlaps the predecessor's tail.

    // first weight row of this CTA's tile(s)
    const int f0 = (EPI == SLAB_SWIGLU) ? (2 * slab + pr) * 64 : (2 * slab + pr) * 128;

    if (warp == 0) {
        // ================= TMA producer (the whole warp runs the loop, one lane issues) =================
        const bool elected = elect_one();
        auto load_w = [&](int stage, int kb, uint32_t full_leader) {
            uint8_t* sW = smem + stage * g.stage_bytes;
            if (leader) mbar_arrive_expect_tx(&full_bar[stage], 2 * g.stage_bytes);
            if (EPI == SLAB_SWIGLU) {
                // 64 gate rows, then the 64 up rows of the same output features
                tma_load_2d_pair(sW, &tmW, full_leader, kb * kBK, f0);
                tma_load_2d_pair(sW + 64 * 128, &tmW, full_leader, kb * kBK, p.N / 2 + f0);
            } else {
                tma_load_2d_pair(sW, &tmW, full_leader, kb * kBK, f0);
            }
        };
        auto load_x = [&](int stage, int kb, uint32_t full_leader) {
            // this CTA's half of every accumulator's token tile
            uint8_t* sX = smem + stage * g.stage_bytes + 128 * 128;
            tma_load_2d_pair(sX, &tmX, full_leader, kb * kBK, pr * h0);
            if (h1) tma_load_2d_pair(sX + h0 * 128, &tmX1, full_leader, kb * kBK, g.n0 + pr * h1);
        };
        const int n_pre = min(stages, kb1 - kb0);
        if (elected)
            for (int i = 0; i < n_pre; ++i) load_w(i, kb0 + i, mapa_u32(&full_bar[i], leader_rank));
        __syncwarp();
        grid_dependency_wait();
        if (lane == 0) SLAB_TRACE(1);
        if (elected)
            for (int i = 0; i < n_pre; ++i) load_x(i, kb0 + i, mapa_u32(&full_bar[i], leader_rank));
        __syncwarp();
        int stage = 0;
        uint32_t phase = 1;                   // the ring has been filled once
        for (int kb = kb0 + n_pre; kb < kb1; ++kb) {
            if (!mbar_wait(&empty_bar[stage], phase ^ 1, abortp)) break;
            const uint32_t full_leader = mapa_u32(&full_bar[stage], leader_rank);
            if (elected) {
                load_w(stage, kb, full_leader);
                load_x(stage, kb, full_leader);
            }
            __syncwarp();
            if (++stage == stages) { stage = 0; phase ^= 1; }
        }
    } else if (warp == 1) {
        // ================= MMA issuer (even CTA of the pair; the whole warp runs the loop, one lane issues) ======
        if (leader) {
            const bool elected = elect_one();
            const uint32_t idesc0 = umma_idesc_bf16(256, g.n0), idesc1 = umma_idesc_bf16(256, g.n1);
            const uint16_t pair_mask = (uint16_t)(0x3u << leader_rank);
            // The operand descriptors of a stage differ from those of stage 0 only in the 16-byte-granular
            // address field, so they are built once and advanced by additions (the field never carries:
            // addresses stay below 256 KB).
            const uint64_t wd0 = umma_desc_k128(smem_u32(smem));
            const uint64_t xd0 = wd0 + ((128 * 128) >> 4);
            const uint32_t stage_units = (uint32_t)g.stage_bytes >> 4, acc_units = (uint32_t)(h0 * 128) >> 4;
            const uint32_t d0 = tmem_base, d1 = tmem_base + g.n0;
            const bool two = g.n_acc == 2;
            int stage = 0;
            uint32_t phase = 0, accum = 0;
            uint64_t wd = wd0, xd = xd0;
            bool ok = true;
#ifdef JOT_SLAB_TRACE
            long long waited = 0;
            const long long loop_c0 = clock64();
#endif
            for (int kb = kb0; kb < kb1; ++kb) {
#ifdef JOT_SLAB_TRACE
                const long long c0 = clock64();
#endif
                if (!mbar_wait(&full_bar[stage], phase, abortp)) { ok = false; break; }
#ifdef JOT_SLAB_TRACE
                waited += clock64() - c0;
                if (kb == kb0 && lane == 0) SLAB_TRACE(2);
#endif
                tc_fence_after();
                if (elected) {
                    if (two) {
#pragma unroll
                        for (int k = 0; k < kBK / 16; ++k) {
                            umma_bf16_pair(d0, wd + 2 * k, xd + 2 * k, idesc0, accum | k);
                            umma_bf16_pair(d1, wd + 2 * k, xd + acc_units + 2 * k, idesc1, accum | k);
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < kBK / 16; ++k) umma_bf16_pair(d0, wd + 2 * k, xd + 2 * k, idesc0, accum | k);
                    }
                    umma_commit_pair(&empty_bar[stage], pair_mask);
                }
                __syncwarp();
                accum = 1;
                wd += stage_units;
                xd += stage_units;
                if (++stage == stages) { stage = 0; phase ^= 1; wd = wd0; xd = xd0; }
            }
            if (ok && elected) umma_commit_pair(&acc_full, pair_mask);
            __syncwarp();
            if (lane == 0) {
                SLAB_TRACE(3);
#ifdef JOT_SLAB_TRACE
                SLAB_TRACE_VAL(4, (unsigned long long)waited);
                SLAB_TRACE_VAL(8, (unsigned long long)(clock64() - loop_c0));
#endif
            }
        }
    }
    __syncwarp();

    // ================= after the main loop =================
    const bool epi_warp = warp >= 2;
    const int quad = warp & 3, grp = (warp - 2) >> 2;          // TMEM lane quadrant; warp group 0 / 1
    const int f_in = quad * 32 + lane;                         // feature row inside the CTA's tile = TMEM lane
    const uint32_t lane_base = tmem_base + (uint32_t(quad * 32) << 16);
    const bool have_acc = kb1 > kb0;                           // a pair with an empty K range contributes zeros
    const int c_lo = (split > 1) ? ks * g.cpo : 0;             // the chunks this CTA writes out
    const int c_hi = (split > 1) ? min(g.n_chunks, c_lo + g.cpo) : g.n_chunks;
    bool ok = true;

    // SLAB_STORE read-out: item i of a thread is (token, 8-column group) = ((f_in + 128 i) / 16, (f_in + 128 i) % 16)
    // of the chunk; the residual of a chunk's four items is requested a whole chunk ahead
    uint4 res[4];
    auto load_residual = [&](int c) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int item = f_in + 128 * i, t = c * 32 + (item >> 4), oc = f0 + (item & 15) * 8;
            res[i] = (t < p.M && oc < p.N) ? *reinterpret_cast<const uint4*>(p.residual + (size_t)t * p.ldc + oc)
                                           : make_uint4(0, 0, 0, 0);
        }
    };
    // SLAB_QKV read-out: 32 tokens x (128 / hd heads) x (hd / 16 groups of 8 rotation pairs) = 256 items per chunk,
    // two per thread; their (cos, sin) rows are requested a whole chunk ahead as well
    float4 rope[2][4];
    auto rope_item = [&](int i, int& tok, int& hh, int& gq) {
        const int groups = p.hd >> 4, heads_here = 128 / p.hd, item = f_in + 128 * i;
        gq = item % groups;
        hh = (item / groups) % heads_here;
        tok = item / (groups * heads_here);
    };
    auto load_rope = [&](int c) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            int tok, hh, gq;
            rope_item(i, tok, hh, gq);
            const int t = c * 32 + tok;
            if (t < p.M) {
                const int seq = t / p.rows_per_seq, pos = p.pos0 + (t - seq * p.rows_per_seq);
                const float4* cs4 = reinterpret_cast<const float4*>(p.rope_cs + (size_t)pos * (p.hd >> 1) + gq * 8);
#pragma unroll
                for (int j = 0; j < 4; ++j) rope[i][j] = cs4[j];
            }
        }
    };
    if (epi_warp) {
        grid_dependency_wait();
        if (EPI == SLAB_STORE && p.residual && c_lo + grp < c_hi) load_residual(c_lo + grp);   // in flight during the main loop
        if (EPI == SLAB_QKV && c_lo + grp < c_hi) load_rope(c_lo + grp);
        if (have_acc) ok = mbar_wait(&acc_full, 0, abortp);
        tc_fence_after();
        if (threadIdx.x == 64) SLAB_TRACE(5);
    }
    float* recv = reinterpret_cast<float*>(smem);              // [split - 1][cpo * 32 tokens][128 features]
    float* stage_buf = reinterpret_cast<float*>(smem + g.recv_bytes) + grp * 2 * (32 * 128);   // two chunk buffers

    auto load_chunk = [&](int c, float* v) {                   // issue only; tmem_ld_wait() before use
        if (have_acc && ok) {
            tmem_ld32(lane_base + c * 32, v);
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0.f;
        }
    };

    if (split > 1) {
        cluster_sync_all();                   // every pair's accumulators are complete, every pipeline is idle
        if (threadIdx.x == 64) SLAB_TRACE(9);
        if (epi_warp) {
            // reduce-scatter: the chunks another pair owns go to the CTA of the same parity in that pair; a warp's
            // store covers 32 consecutive features of one token, 128 contiguous bytes (strided 16-byte stores
            // of one feature's tokens were measured at half the speed)
            for (int c = grp; c < g.n_chunks; c += 2) {
                const int q = c / g.cpo;
                if (q == ks) continue;
                float v[32];
                load_chunk(c, v);
                tmem_ld_wait_regs(v);
                const int slot = ks < q ? ks : ks - 1;
                float* dst = recv + ((size_t)(slot * g.cpo + (c - q * g.cpo)) * 32) * 128 + f_in;
                const uint32_t remote = mapa_u32(dst, (uint32_t)(2 * q + pr));
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote + j * 512), "f"(v[j]) : "memory");
            }
        }
        if (threadIdx.x == 64) SLAB_TRACE(10);
        cluster_sync_all();                   // release / acquire: the partial sums have landed
        if (threadIdx.x == 64) SLAB_TRACE(6);
    }

    if (epi_warp) {
        // this pair's own partial sum takes its place in the fixed order s = 0 .. split-1
        auto reduce_chunk = [&](int c, float* v) {
            float acc[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) acc[j] = 0.f;
            for (int s = 0; s < split; ++s) {
                if (s == ks) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[j] += v[j];
                } else {
                    const float* r = recv + ((size_t)((s < ks ? s : s - 1) * g.cpo + (c - c_lo)) * 32) * 128 + f_in;
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[j] += r[j * 128];
                }
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = acc[j];
        };
        const int tid_g = f_in;                                 // 0..127 inside the warp group
        const uint32_t bar_id = 1 + grp;
        float v[32], vn[32];
        if (c_lo + grp < c_hi) load_chunk(c_lo + grp, v);
        int it = 0;
        tmem_ld_wait_regs(v);
        for (int c = c_lo + grp; c < c_hi; c += 2, ++it) {
            const bool more = c + 2 < c_hi;
            if (more) load_chunk(c + 2, vn);                    // the next chunk's accumulators travel meanwhile
            if (split > 1) reduce_chunk(c, v);
            const int t0 = c * 32;                              // first token (input row) of the chunk
            {
                float* sb = stage_buf + (it & 1) * (32 * 128);
                bool staged = true;
                if (EPI == SLAB_QKV) {
                    const int head = (f0 + f_in) / p.hd;
                    if (head >= p.nq + p.nkv) {
                        // V head: this thread's 32 tokens of feature d are consecutive keys of row d of V^T
                        staged = false;
                        const int kvh = head - p.nq - p.nkv, dd = (f0 + f_in) % p.hd;
                        if (f0 + f_in < p.N) {
                            const int seq0 = t0 / p.rows_per_seq, pos_first = p.pos0 + (t0 - seq0 * p.rows_per_seq);
                            const bool one_seq = (t0 + 31) / p.rows_per_seq == seq0 && t0 + 31 < p.M;
                            __nv_bfloat16* row = p.vt + ((size_t)(seq0 * p.nkv + kvh) * p.hd + dd) * p.Lp + pos_first;
                            if (one_seq && (pos_first & 7) == 0) {
#pragma unroll
                                for (int q4 = 0; q4 < 4; ++q4) {
                                    uint4 ov;
                                    __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
                                    for (int j = 0; j < 4; ++j) o2[j] = __floats2bfloat162_rn(v[q4 * 8 + 2 * j], v[q4 * 8 + 2 * j + 1]);
                                    *reinterpret_cast<uint4*>(row + q4 * 8) = ov;
                                }
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j) {
                                    const int t = t0 + j;
                                    if (t < p.M) {
                                        const int seq = t / p.rows_per_seq, pos = p.pos0 + (t - seq * p.rows_per_seq);
                                        p.vt[((size_t)(seq * p.nkv + kvh) * p.hd + dd) * p.Lp + pos] = __float2bfloat16_rn(v[j]);
                                    }
                                }
                            }
                        }
                    }
                }
                if (staged) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) sb[j * 128 + f_in] = v[j];
                }
                if (threadIdx.x == 64 && it == 0) SLAB_TRACE(11);
                asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
                if (threadIdx.x == 64 && it == 0) SLAB_TRACE(12);
                // ---- token-major read-out of the 32 x 128 chunk, 16-byte stores ----
                if (EPI == SLAB_STORE) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int item = tid_g + 128 * i, tok = item >> 4, gq = item & 15, t = t0 + tok, oc = f0 + gq * 8;
                        if (t >= p.M || oc >= p.N) continue;
                        const float4 a = *reinterpret_cast<const float4*>(sb + tok * 128 + gq * 8);
                        const float4 b = *reinterpret_cast<const float4*>(sb + tok * 128 + gq * 8 + 4);
                        float x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
                        if (p.residual) {
                            const __nv_bfloat162* r2 = reinterpret_cast<const __nv_bfloat162*>(&res[i]);
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
                        *reinterpret_cast<uint4*>(p.C + (size_t)t * p.ldc + oc) = ov;
                    }
                    if (p.residual && more) load_residual(c + 2);
                } else if (EPI == SLAB_SWIGLU) {
                    const int n_out = p.N / 2;
#pragma unroll 1
                    for (int item = tid_g; item < 32 * 8; item += 128) {
                        const int tok = item >> 3, gq = item & 7, t = t0 + tok, oc = f0 + gq * 8;
                        if (t >= p.M || oc >= n_out) continue;
                        const float* gp = sb + tok * 128 + gq * 8;
                        const float4 g0 = *reinterpret_cast<const float4*>(gp), g1 = *reinterpret_cast<const float4*>(gp + 4);
                        const float4 u0 = *reinterpret_cast<const float4*>(gp + 64), u1 = *reinterpret_cast<const float4*>(gp + 68);
                        const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
                        const float uu[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
                        uint4 ov;
                        __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float a0 = gg[2 * j] / (1.f + __expf(-gg[2 * j])) * uu[2 * j];
                            const float a1 = gg[2 * j + 1] / (1.f + __expf(-gg[2 * j + 1])) * uu[2 * j + 1];
                            o2[j] = __floats2bfloat162_rn(a0, a1);
                        }
                        *reinterpret_cast<uint4*>(p.C + (size_t)t * p.ldc + oc) = ov;
                    }
                } else {
                    // Q and K heads: pairs (j, j + hd/2) of one head, 8 pairs per item
                    const int hd = p.hd, half = hd >> 1;
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        int tok, hh, gq;
                        rope_item(i, tok, hh, gq);
                        const int t = t0 + tok, oc = f0 + hh * hd + gq * 8;
                        const int head = oc / hd;
                        if (t >= p.M || oc >= p.N || head >= p.nq + p.nkv) continue;
                        const int seq = t / p.rows_per_seq, pos = p.pos0 + (t - seq * p.rows_per_seq);
                        const float* lp = sb + tok * 128 + hh * hd + gq * 8;
                        const float4 l0 = *reinterpret_cast<const float4*>(lp), l1 = *reinterpret_cast<const float4*>(lp + 4);
                        const float4 x0h = *reinterpret_cast<const float4*>(lp + half), x1h = *reinterpret_cast<const float4*>(lp + half + 4);
                        const float lo[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
                        const float hi[8] = {x0h.x, x0h.y, x0h.z, x0h.w, x1h.x, x1h.y, x1h.z, x1h.w};
                        uint4 olo, ohi;
                        __nv_bfloat162* l2 = reinterpret_cast<__nv_bfloat162*>(&olo);
                        __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&ohi);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float4 k = rope[i][j];              // (cos, sin) of pairs 2j and 2j + 1
                            // the projection's output is bf16; the rotation acts on the rounded values
                            const float2 x0 = __bfloat1622float2(__floats2bfloat162_rn(lo[2 * j], lo[2 * j + 1]));
                            const float2 x1 = __bfloat1622float2(__floats2bfloat162_rn(hi[2 * j], hi[2 * j + 1]));
                            l2[j] = __floats2bfloat162_rn(x0.x * k.x - x1.x * k.y, x0.y * k.z - x1.y * k.w);
                            h2[j] = __floats2bfloat162_rn(x1.x * k.x + x0.x * k.y, x1.y * k.z + x0.y * k.w);
                        }
                        __nv_bfloat16* dlo = p.C + ((size_t)seq * p.L + pos) * p.ldc + oc;
                        *reinterpret_cast<uint4*>(dlo) = olo;
                        *reinterpret_cast<uint4*>(dlo + half) = ohi;
                    }
                    if (more) load_rope(c + 2);
                }
            }
            if (threadIdx.x == 64 && it == 0) SLAB_TRACE(13);
            if (more) {
                tmem_ld_wait_regs(vn);
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = vn[j];
            }
        }
    }

    if (threadIdx.x == 64) SLAB_TRACE(7);
    // ---- teardown: nobody leaves while a CTA of the cluster may still signal or write across ----
    tc_fence_before();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, tmem_cols);
    }
    if (threadIdx.x == 0 && abort_flag && p.status) atomicExch(p.status, 4);
}


// ---------------------------------------------------------------------------------------------------------------
// Gate/up projection + SwiGLU for canvases of 353 .. 384 rows: two units of work per CTA pair, one launch.
//
// With S pair-slabs and P pairs on the device (96 and 74 for d_ff = 12288 on 148 SMs) one slab per pair leaves slabs
// over, and cutting those along K needs a second launch, a reduce-scatter and an epilogue that nothing overlaps.
// Here A = S - B pairs each take ONE WHOLE slab (all tokens: accumulators of 256 + 128 token columns), and then one of
// the remaining B = S / 4 slabs for ONE THIRD of the tokens (128 token columns, full K): 3 B <= A second units, no
// partial sums anywhere.  The second unit's accumulator is a third region of tensor memory (256 + 128 + 128 = 512
// columns), so the first unit's epilogue runs under the second unit's main loop.  Its four chunk buffers are the last
// 16 KB of the first four pipeline stages: a second-unit stage holds 16 KB of W and 8 KB of tokens and leaves exactly
// that much of its 40 KB unused.  Weights of a second-unit slab are read by three pairs, at about the same time: from
// HBM once.
constexpr int kSlab2Stages = 5;
constexpr int kSlab2StageBytes = 128 * 128 + 192 * 128;         // W tile + this CTA's half of 384 tokens
constexpr int kSlab2Smem = kSlab2Stages * kSlab2StageBytes + 1024;

struct Slab2Plan {
    int A, B, G;        // pairs (= first units), second-unit slabs, token groups of 128 per second-unit slab
    bool ok;
};
#ifndef JOT_SLAB_TWO_UNITS
#define JOT_SLAB_TWO_UNITS 1
#endif
__host__ __device__ inline Slab2Plan slab2_plan(int M, int n_slabs, int pairs) {
    Slab2Plan q{0, 0, 3, false};
    if (!JOT_SLAB_TWO_UNITS) return q;
    if (M <= 352 || M > 384) return q;             // accumulators of exactly 256 + 128 token columns
    q.B = n_slabs / (q.G + 1);
    q.A = n_slabs - q.B;
    q.ok = q.B > 0 && q.A <= pairs && q.G * q.B <= q.A;
    return q;
}

__global__ void __launch_bounds__(kSlabThreads, 1)
gemm_slab_gateup2_kernel(const GemmParams p, const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                         const __grid_constant__ CUtensorMap tmX1) {
    constexpr int STAGES = kSlab2Stages, STAGE_BYTES = kSlab2StageBytes;
    constexpr int EPI = SLAB_SWIGLU;          // (for the trace points of instrumented builds)
    (void)EPI;
    constexpr int N0 = 256, N1 = 128, H0 = N0 / 2, H1 = N1 / 2;      // token columns per accumulator; rows a CTA loads
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], acc_full[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                    // 0 / 1
    const int pr = (int)(rank & 1u);
    const bool leader = pr == 0;
    const int pair = (int)(blockIdx.x >> 1);
    const int n_slabs = p.N / 256, A = p.slab0, G = p.slab_split, B = n_slabs - A;
    // unit 0: slab `pair`, every token; unit 1 (pairs below G * B): slab A + pair / G, tokens [128 (pair % G), + 128)
    const int n_units = pair < G * B ? 2 : 1;
    const int slab_of[2] = {pair, A + pair / G};
    const int tok1 = (pair % G) * 128;
    const int num_kb = (p.K + kBK - 1) / kBK;
    const int total = n_units * num_kb;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        mbar_init(&acc_full[0], 1);
        mbar_init(&acc_full[1], 1);
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmX);
        tma_prefetch_desc(&tmX1);
    }
    if (warp == 1) {
        tmem_alloc_pair(&tmem_base_slot, 512);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    cluster_sync_all();                       // the pair's barriers exist before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    if (threadIdx.x == 0) SLAB_TRACE(0);
    grid_launch_dependents();
    auto f0_of = [&](int u) { return (2 * slab_of[u] + pr) * 64; };     // first gate row (= output column) of this CTA's tile

    if (warp == 0) {
        // ================= TMA producer (the whole warp runs the loop, one lane issues) =================
        const bool elected = elect_one();
        auto load_w = [&](int stage, int i, uint32_t full_leader) {
            const int u = i >= num_kb, kb = i - u * num_kb, f0 = f0_of(u);
            uint8_t* sW = smem + stage * STAGE_BYTES;
            if (leader) mbar_arrive_expect_tx(&full_bar[stage], u ? 2 * (128 * 128 + H1 * 128) : 2 * STAGE_BYTES);
            tma_load_2d_pair(sW, &tmW, full_leader, kb * kBK, f0);                          // 64 gate rows
            tma_load_2d_pair(sW + 64 * 128, &tmW, full_leader, kb * kBK, p.N / 2 + f0);     // the matching 64 up rows
        };
        auto load_x = [&](int stage, int i, uint32_t full_leader) {
            const int u = i >= num_kb, kb = i - u * num_kb;
            uint8_t* sX = smem + stage * STAGE_BYTES + 128 * 128;
            if (u == 0) {
                tma_load_2d_pair(sX, &tmX, full_leader, kb * kBK, pr * H0);
                tma_load_2d_pair(sX + H0 * 128, &tmX1, full_leader, kb * kBK, N0 + pr * H1);
            } else {
                tma_load_2d_pair(sX, &tmX1, full_leader, kb * kBK, tok1 + pr * H1);
            }
        };
        // the first W tiles go out before the wait on the preceding kernel (weights are nobody's output)
        const int n_pre = min(STAGES, total);
        if (elected)
            for (int i = 0; i < n_pre; ++i) load_w(i, i, mapa_u32(&full_bar[i], 0));
        __syncwarp();
        grid_dependency_wait();
        if (lane == 0) SLAB_TRACE(1);
        if (elected)
            for (int i = 0; i < n_pre; ++i) load_x(i, i, mapa_u32(&full_bar[i], 0));
        __syncwarp();
        int stage = 0;
        uint32_t phase = 1;                   // the ring has been filled once
        for (int i = n_pre; i < total; ++i) {
            if (!mbar_wait(&empty_bar[stage], phase ^ 1, abortp)) break;
            const uint32_t full_leader = mapa_u32(&full_bar[stage], 0);
            if (elected) {
                load_w(stage, i, full_leader);
                load_x(stage, i, full_leader);
            }
            __syncwarp();
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
    } else if (warp == 1) {
        // ================= MMA issuer (even CTA of the pair; the whole warp runs the loop, one lane issues) ======
        if (leader) {
            const bool elected = elect_one();
            const uint32_t idesc0 = umma_idesc_bf16(256, N0), idesc1 = umma_idesc_bf16(256, N1);
            const uint16_t pair_mask = 0x3u;
            const uint64_t wd0 = umma_desc_k128(smem_u32(smem));
            const uint64_t xd0 = wd0 + ((128 * 128) >> 4);
            constexpr uint32_t stage_units = (uint32_t)STAGE_BYTES >> 4, acc_units = (uint32_t)(H0 * 128) >> 4;
            int stage = 0;
            uint32_t phase = 0;
            uint64_t wd = wd0, xd = xd0;
            bool ok = true;
            for (int u = 0; ok && u < n_units; ++u) {
                uint32_t accum = 0;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&full_bar[stage], phase, abortp)) { ok = false; break; }
                    if (u == 0 && kb == 0 && lane == 0) SLAB_TRACE(2);
                    tc_fence_after();
                    if (elected) {
                        if (u == 0) {
#pragma unroll
                            for (int k = 0; k < kBK / 16; ++k) {
                                umma_bf16_pair(tmem_base, wd + 2 * k, xd + 2 * k, idesc0, accum | k);
                                umma_bf16_pair(tmem_base + N0, wd + 2 * k, xd + acc_units + 2 * k, idesc1, accum | k);
                            }
                        } else {
#pragma unroll
                            for (int k = 0; k < kBK / 16; ++k)
                                umma_bf16_pair(tmem_base + N0 + N1, wd + 2 * k, xd + 2 * k, idesc1, accum | k);
                        }
                        umma_commit_pair(&empty_bar[stage], pair_mask);
                    }
                    __syncwarp();
                    accum = 1;
                    wd += stage_units;
                    xd += stage_units;
                    if (++stage == STAGES) { stage = 0; phase ^= 1; wd = wd0; xd = xd0; }
                }
                if (ok && elected) umma_commit_pair(&acc_full[u], pair_mask);
                __syncwarp();
                if (lane == 0) SLAB_TRACE(3 + u);
            }
        }
    } else {
        // ================= epilogue: warps 2..9, two warps per TMEM lane quadrant (a lane is an output FEATURE) =======
        const int quad = warp & 3, grp = (warp - 2) >> 2;
        const int f_in = quad * 32 + lane;
        const uint32_t lane_base = tmem_base + (uint32_t(quad * 32) << 16);
        // chunk buffer i of the group = bytes [24 KB, 40 KB) of pipeline stage 2 grp + i: free once unit 0's products
        // have retired (unit 1's loads fill only the first 24 KB of a stage; a pair without a second unit loads nothing)
        auto chunk_buf = [&](int i) { return reinterpret_cast<float*>(smem + (2 * grp + i) * STAGE_BYTES + 24 * 1024); };
        const uint32_t bar_id = 1 + grp;
        const int n_out = p.N / 2;
        grid_dependency_wait();
        int it = 0;
        for (int u = 0; u < n_units; ++u) {
            // (the tensor-memory loads below are warp-wide: a warp gives up as one)
            if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[u], 0, abortp))) break;
            tc_fence_after();
            if (threadIdx.x == 64) SLAB_TRACE(5 + 2 * u);
            const int f0 = f0_of(u);
            const int n_ch = u ? N1 / 32 : (N0 + N1) / 32;                    // 32-token chunks of this unit
            const uint32_t col0 = u ? N0 + N1 : 0;                            // its first accumulator column
            const int tok0 = u ? tok1 : 0;                                     // its first token
            float v[32], vn[32];
            if (grp < n_ch) tmem_ld32(lane_base + col0 + grp * 32, v);
            tmem_ld_wait_regs(v);
            for (int c = grp; c < n_ch; c += 2, ++it) {
                const bool more = c + 2 < n_ch;
                if (more) tmem_ld32(lane_base + col0 + (c + 2) * 32, vn);     // the next chunk's accumulators travel meanwhile
                const int t0 = tok0 + c * 32;
                float* sb = chunk_buf(it & 1);
#pragma unroll
                for (int j = 0; j < 32; ++j) sb[j * 128 + f_in] = v[j];
                asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
                // token-major read-out of the 32 x 128 chunk (64 gate + 64 up features per token), 16-byte stores
#pragma unroll 1
                for (int item = f_in; item < 32 * 8; item += 128) {
                    const int tok = item >> 3, gq = item & 7, t = t0 + tok, oc = f0 + gq * 8;
                    if (t >= p.M || oc >= n_out) continue;
                    const float* gp = sb + tok * 128 + gq * 8;
                    const float4 g0 = *reinterpret_cast<const float4*>(gp), g1 = *reinterpret_cast<const float4*>(gp + 4);
                    const float4 u0 = *reinterpret_cast<const float4*>(gp + 64), u1 = *reinterpret_cast<const float4*>(gp + 68);
                    const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
                    const float uu[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
                    uint4 ov;
                    __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float a0 = gg[2 * j] / (1.f + __expf(-gg[2 * j])) * uu[2 * j];
                        const float a1 = gg[2 * j + 1] / (1.f + __expf(-gg[2 * j + 1])) * uu[2 * j + 1];
                        o2[j] = __floats2bfloat162_rn(a0, a1);
                    }
                    *reinterpret_cast<uint4*>(p.C + (size_t)t * p.ldc + oc) = ov;
                }
                if (more) {
                    tmem_ld_wait_regs(vn);
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = vn[j];
                }
            }
            if (threadIdx.x == 64) SLAB_TRACE(6 + 2 * u);
        }
    }
    __syncwarp();

    // ---- teardown: nobody leaves while the other CTA of the pair may still signal or read across ----
    tc_fence_before();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, 512);
    }
    if (threadIdx.x == 0 && abort_flag && p.status) atomicExch(p.status, 4);
}

}  // namespace jot
