// Bidirectional (unmasked) grouped-query softmax attention on tcgen05 / tensor memory, fed by TMA.
//
// Persistent CTAs walk over work items (query block of 128 rows, query head, sequence), ordered so that the
// CTAs running side by side share K and V of one KV head in L2.  For one item the keys are visited ONCE, in
// blocks of 128:
//   S = Q K^T for the block (tensor memory, double buffered: S(j+1) is computed while block j is in softmax)
//   P = bf16(exp((S - m_ref) / sqrt(hd))) written back INTO the score buffer (each thread replaces scores it has just
//       read) and used from there as the A operand of  O += P V : P never touches shared memory, whose bandwidth the
//       MMAs with both operands in shared memory already take whole
// Two threads share a query row, each owning 64 of the block's 128 key columns, and each keeps ITS OWN running
// reference maximum m_ref, row sum and output accumulator (O_left and O_right in tensor memory, fed by the two
// 64-key halves of P V): no exchange between the two threads per block, only once per item, when the halves
// are combined as (O_l 2^(m_l - m) + O_r 2^(m_r - m)) / (l_l 2^(m_l - m) + l_r 2^(m_r - m)).
// The reference maximum is lazy: it is raised only when a block's maximum exceeds it by more than 2^8
// (probabilities up to 256 are exact enough in bf16 and fp32); the owner thread then rescales its row of its
// accumulator in tensor memory (tcgen05.ld / st, once the P V of the previous block has retired) and its running
// sum.  With well-behaved scores that happens in the first block only, where there is nothing to rescale.
// Nothing makes a softmax warp wait for the previous P V otherwise, so a warp may run one block ahead of another:
// barriers that count warp arrivals exist once per score buffer.
// The combined output tile is staged in shared memory and leaves as whole rows.
//
//   warp 0 (one lane)  TMA producer: Q per item, then K and V^T block by block
//   warp 1             MMA issuer (the whole warp runs the loop, one elected lane issues)
//   warps 2..9         softmax: thread (r, hf) owns query row r (TMEM lane) and key columns [64 hf, 64 hf + 64)
//
// Layouts: qkv [B*L, (nq + 2 nkv) * hd] after RoPE (3-D tensor map (col, position, sequence) so that a
// block never reads across a sequence boundary: out-of-range positions read as zero); V transposed
// vt [B * nkv * hd, Lp] with keys contiguous, so that both products take K-major operands.
#pragma once
#include "pdl.cuh"
#include "ptx.cuh"

namespace jot {

constexpr int kAttnThreads = 320;          // producer warp, MMA warp, 8 softmax warps
constexpr int kAttnSoftmaxThreads = 256;

struct AttnParams {
    int B, L, nq, nkv;
    float scale_log2e;            // log2(e) / sqrt(hd)
    __nv_bfloat16* out;           // [B*q_cnt, nq*hd]: row b * q_cnt + (q - q_lo)
    int32_t* status;
    // queries are canvas positions q_lo .. q_lo + q_cnt - 1 of every sequence (the whole canvas: 0, L; one block
    // of a block-wise KV cache: its rows only); keys and values are always all L positions
    int q_lo, q_cnt;
};

template <int HD>
struct AttnSmem {
    static constexpr int KB = HD / 64;                    // 64-wide sub-tiles along the head dimension
    static constexpr int Q_BYTES = KB * 128 * 128;        // 128 rows x 128 B per sub-tile
    static constexpr int K_BYTES = KB * 128 * 128;
    static constexpr int V_BYTES = 2 * HD * 128;          // two 64-key sub-tiles of HD rows
    static constexpr int O_BYTES = 128 * HD * 2;          // one output tile, staged for the copy-out
    static constexpr int DYN_BYTES = Q_BYTES + 2 * K_BYTES + 2 * V_BYTES + O_BYTES + 1024;
};

#ifdef JOT_ATTN_TRACE
// Cycles one softmax thread of every CTA spent in each phase of the key loop; only in instrumented builds.
__device__ long long g_attn_trace[256 * 16];
#define ATTN_T(var) const long long var = clock64()
#define ATTN_ACC(slot, a, b) do { if (threadIdx.x == 64) g_attn_trace[(blockIdx.x & 255) * 16 + (slot)] += (b) - (a); } while (0)
#else
#define ATTN_T(var) do { } while (0)
#define ATTN_ACC(slot, a, b) do { } while (0)
#endif

template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tmQKV, const __grid_constant__ CUtensorMap tmVt) {
    using SM = AttnSmem<HD>;
    constexpr int KB = SM::KB;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC_S = umma_idesc_bf16(128, 128);
    constexpr uint32_t IDESC_O = umma_idesc_bf16(128, HD);
    constexpr uint32_t O_COL = 256;            // S buffers at columns 0 and 128, O_left at 256, O_right at 384
    constexpr float kRaise = 8.f;              // the reference maximum follows a block maximum more than 2^8 above it

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + SM::Q_BYTES;          // 2 stages
    uint8_t* sV = sK + 2 * SM::K_BYTES;      // 2 stages
    uint8_t* sO = sV + 2 * SM::V_BYTES;
    __shared__ uint64_t q_full, q_empty, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], p_full[2],
        o_full, o_empty, x_bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ float x_max[2][2][128], x_sum[2][2][128];      // [item parity][half][row]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int L = p.L;
    const int nkb = (L + 127) / 128, nqb = (p.q_cnt + 127) / 128;
    const int group = p.nq / p.nkv;
    const int n_items = p.B * p.nq * nqb;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&q_full, 1);
        mbar_init(&q_empty, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&k_full[i], 1);
            mbar_init(&k_empty[i], 1);
            mbar_init(&v_full[i], 1);
            mbar_init(&v_empty[i], 1);
            mbar_init(&s_full[i], 1);
            mbar_init(&p_full[i], kAttnSoftmaxThreads / 32);      // one arrival per softmax warp
        }
        mbar_init(&o_full, 1);
        mbar_init(&o_empty, 8);
        mbar_init(&x_bar, kAttnSoftmaxThreads / 32);
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmQKV);
        tma_prefetch_desc(&tmVt);
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
    grid_launch_dependents();
    grid_dependency_wait();

    // item -> (query block, head, sequence); query blocks fastest, then the heads of one KV group
    auto decode = [&](int item, int& q_blk, int& h, int& b) {
        q_blk = item % nqb;
        const int t = item / nqb;
        h = t % p.nq;
        b = t / p.nq;
    };

    if (warp == 0) {
        if (lane == 0) {
            uint32_t g = 0;              // running count of key blocks (K and V loads, S and P.V products)
            int it = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++it) {
                int q_blk, h, b;
                decode(item, q_blk, h, b);
                const int kvh = h / group;
                const int q_col = h * HD, k_col = (p.nq + kvh) * HD, vt_row = (b * p.nkv + kvh) * HD;
                if (!mbar_wait(&q_empty, (it & 1) ^ 1, abortp)) break;
                mbar_arrive_expect_tx(&q_full, SM::Q_BYTES);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
                    tma_load_3d(sQ + kb * 16384, &tmQKV, &q_full, q_col + kb * 64, p.q_lo + q_blk * 128, b);
                for (int j = 0; j < nkb; ++j, ++g) {
                    const int st = g & 1;
                    if (!mbar_wait(&k_empty[st], ((g >> 1) & 1) ^ 1, abortp)) { ok = false; break; }
                    mbar_arrive_expect_tx(&k_full[st], SM::K_BYTES);
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb)
                        tma_load_3d(sK + st * SM::K_BYTES + kb * 16384, &tmQKV, &k_full[st], k_col + kb * 64, j * 128, b);
                    if (!mbar_wait(&v_empty[st], ((g >> 1) & 1) ^ 1, abortp)) { ok = false; break; }
                    mbar_arrive_expect_tx(&v_full[st], SM::V_BYTES);
#pragma unroll
                    for (int half = 0; half < 2; ++half)
                        tma_load_2d(sV + st * SM::V_BYTES + half * (HD * 128), &tmVt, &v_full[st], j * 128 + half * 64, vt_row);
                }
            }
        }
    } else if (warp == 1) {
        // MMA issuer.  The whole warp runs the loop and one elected lane issues: a loop entered by one lane alone turns
        // every operand descriptor into a per-thread value that has to be made uniform again for each instruction,
        // which costs more than the instruction itself.
        const bool elected = elect_one();
        auto wait_warp = [&](uint64_t* bar, uint32_t parity) -> bool {
            const bool w = mbar_wait(bar, parity, abortp);
            return __all_sync(0xffffffffu, w);
        };
        const uint64_t qd = umma_desc_k128(smem_u32(sQ)), kd0 = umma_desc_k128(smem_u32(sK));
        const uint64_t vd0 = umma_desc_k128(smem_u32(sV));
        uint32_t gs = 0, gv = 0;     // S products and P.V products issued so far
        int it = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++it) {
            auto issue_S = [&](bool last) -> bool {
                const int st = gs & 1;
                if (!wait_warp(&k_full[st], (gs >> 1) & 1)) return false;
                // the buffer holds the probabilities of the block two back until their P.V has retired (the barrier
                // that also frees that block's V stage; one barrier per buffer, so that a wait can never be overtaken)
                if (!wait_warp(&v_empty[st], ((gs >> 1) & 1) ^ 1)) return false;
                tc_fence_after();
                if (elected) {
                    const uint64_t kd = kd0 + (uint64_t)(st * (SM::K_BYTES >> 4));
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_bf16(tmem_base + st * 128, qd + kb * 1024 + 2 * k, kd + kb * 1024 + 2 * k, IDESC_S, (kb | k) != 0);
                    umma_commit(&k_empty[st]);
                    umma_commit(&s_full[st]);
                    if (last) umma_commit(&q_empty);          // Q may now be overwritten by the next item's
                }
                __syncwarp();
                ++gs;
                return true;
            };
            auto issue_PV = [&](int j) -> bool {
                const int vs = gv & 1;
                if (!wait_warp(&v_full[vs], (gv >> 1) & 1)) return false;
                if (!wait_warp(&p_full[vs], (gv >> 1) & 1)) return false;
                // the first product of an item overwrites the accumulators: the previous item's output step must be done
                if (j == 0 && !wait_warp(&o_empty, (it & 1) ^ 1)) return false;
                tc_fence_after();
                if (elected) {
                    const uint64_t vd = vd0 + (uint64_t)(vs * (SM::V_BYTES >> 4));
                    // P sits where the block's scores were: the left 64 keys (32 packed columns at the start of the
                    // buffer) feed O_left, the right 64 (32 columns from column 64) feed O_right; 8 columns per MMA
#pragma unroll
                    for (int half = 0; half < 2; ++half)
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_bf16_ts(tmem_base + O_COL + half * 128, tmem_base + vs * 128 + half * 64 + 8 * k,
                                         vd + half * (HD * 8) + 2 * k, IDESC_O, (j | k) != 0);
                    umma_commit(&v_empty[vs]);
                    if (j == nkb - 1) umma_commit(&o_full);
                }
                __syncwarp();
                ++gv;
                return true;
            };
            ok = wait_warp(&q_full, it & 1);
            ok = ok && issue_S(nkb == 1);
            for (int j = 1; ok && j < nkb; ++j) {
                ok = issue_S(j == nkb - 1);
                if (ok) ok = issue_PV(j - 1);
            }
            if (ok) ok = issue_PV(nkb - 1);
        }
    } else {
        // ======== softmax: thread (r, hf) owns row r and key columns [64 hf, 64 hf + 64) of every block ========
        const int quad = warp & 3, hf = (warp - 2) >> 2;
        const int r = quad * 32 + lane;
        const uint32_t lane_base = tmem_base + (uint32_t(quad * 32) << 16);
        const uint32_t o_mine = lane_base + O_COL + hf * 128;      // this thread's row of ITS accumulator
        const float c = p.scale_log2e;
        uint32_t g = 0;
        int it = 0;
        bool ok = true;
        ATTN_T(t_role0);
        // The tensor-memory loads and stores below are warp-wide instructions: the 32 threads of a warp must reach
        // them together.  So every wait is followed by a vote, and a warp leaves the loops as one.
        auto wait_all = [&](uint64_t* bar, uint32_t parity) -> bool {
            const bool w = mbar_wait(bar, parity, abortp);
            return __all_sync(0xffffffffu, w);
        };
        for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++it) {
            int q_blk, h, b;
            decode(item, q_blk, h, b);
            float mc = -INFINITY, l = 0.f;          // reference maximum (scaled to base-2 exponents) and row sum
            for (int j = 0; ok && j < nkb; ++j, ++g) {
                const int st = g & 1;
                ATTN_T(t0);
                if (!wait_all(&s_full[st], (g >> 1) & 1)) { ok = false; break; }
                ATTN_T(t1);
                ATTN_ACC(0, t0, t1);
                tc_fence_after();
                float v[64];
                tmem_ld32(lane_base + st * 128 + hf * 64, v);
                tmem_ld32(lane_base + st * 128 + hf * 64 + 32, v + 32);
                tmem_ld_wait_regs(v);
                tmem_ld_wait_regs(v + 32);
                ATTN_T(t2);
                ATTN_ACC(1, t1, t2);
                const int key0 = j * 128 + hf * 64;
                const bool whole = key0 + 64 <= L;            // every key of this half exists: no per-key bound checks
                float bm = -INFINITY;
                if (whole) {
#pragma unroll
                    for (int t = 0; t < 64; t += 2) bm = fmaxf(bm, fmaxf(v[t], v[t + 1]));
                } else {
#pragma unroll
                    for (int t = 0; t < 64; ++t) bm = (key0 + t < L) ? fmaxf(bm, v[t]) : bm;
                }
                const float bmc = bm * c;
                const bool raise = bmc > mc + kRaise || (mc == -INFINITY && bm > -INFINITY);
                const bool shrink = raise && j > 0 && mc > -INFINITY;       // something accumulated against the old reference
                // where the reference rises, what was accumulated so far shrinks by 2^(old - new); by 1 elsewhere
                const float f = shrink ? ex2_approx(mc - bmc) : 1.f;
                if (raise) mc = bmc;
                l *= f;
                uint32_t packed[32];
                if (whole) {                                  // (mc is finite here: the half has keys)
                    float l0 = 0.f, l1 = 0.f;
#pragma unroll
                    for (int t = 0; t < 32; ++t) {
                        const float e0 = ex2_approx(fmaf(v[2 * t], c, -mc));
                        const float e1 = ex2_approx(fmaf(v[2 * t + 1], c, -mc));
                        l0 += e0;
                        l1 += e1;
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(e0, e1);
                        packed[t] = *reinterpret_cast<uint32_t*>(&h2);
                    }
                    l += l0 + l1;
                } else if (mc > -INFINITY) {
#pragma unroll
                    for (int t = 0; t < 32; ++t) {
                        const float e0 = (key0 + 2 * t < L) ? ex2_approx(fmaf(v[2 * t], c, -mc)) : 0.f;
                        const float e1 = (key0 + 2 * t + 1 < L) ? ex2_approx(fmaf(v[2 * t + 1], c, -mc)) : 0.f;
                        l += e0 + e1;
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(e0, e1);
                        packed[t] = *reinterpret_cast<uint32_t*>(&h2);
                    }
                } else {
#pragma unroll
                    for (int t = 0; t < 32; ++t) packed[t] = 0u;          // no valid key in this half so far
                }
                ATTN_T(t3);
                ATTN_ACC(2, t2, t3);
                if (__any_sync(0xffffffffu, shrink)) {
                    // warp-uniform branch (tensor-memory loads and stores are warp-wide): every thread passes its
                    // accumulator row through, once the previous P.V has retired
                    if (!wait_all(&v_empty[(g - 1) & 1], ((g - 1) >> 1) & 1)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int ch = 0; ch < HD / 32; ++ch) {
                        float o[32];
                        tmem_ld32(o_mine + ch * 32, o);
                        tmem_ld_wait_regs(o);
#pragma unroll
                        for (int t = 0; t < 32; ++t) o[t] *= f;
                        tmem_st32(o_mine + ch * 32, o);
                    }
                }
                ATTN_T(t4);
                ATTN_ACC(3, t3, t4);
                // this thread's 64 probabilities, packed, replace the first 32 of the 64 scores it has just read: row r
                // of the A operand of P.V (K-major: two keys per column), which nobody else reads or writes
                tmem_st32(lane_base + st * 128 + hf * 64, reinterpret_cast<const float*>(packed));
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                // One arrival per warp, on the barrier of THIS buffer: a warp may be a block ahead of another one (nothing
                // makes it wait for the previous P.V any more), and its arrival for the next block must not count here.
                if (lane == 0) mbar_arrive(&p_full[st]);
                ATTN_T(t5);
                ATTN_ACC(4, t4, t5);
                ATTN_ACC(6, t0, t0 + 1);
            }
            if (!ok) break;
            // ---- the two halves of a row meet ----
            ATTN_T(t6);
            // (two sets, by item parity: a warp that is already in the next item must not overwrite what a slower
            // warp has yet to read)
            x_max[it & 1][hf][r] = mc;
            x_sum[it & 1][hf][r] = l;
            __syncwarp();
            if (lane == 0) mbar_arrive(&x_bar);
            if (!wait_all(&x_bar, it & 1)) { ok = false; break; }
            ATTN_T(t6a);
            ATTN_ACC(8, t6, t6a);
            const float mo = x_max[it & 1][hf ^ 1][r], lo = x_sum[it & 1][hf ^ 1][r];
            const float m = fmaxf(mc, mo);
            const float a_me = mc > -INFINITY ? ex2_approx(mc - m) : 0.f;
            const float a_ot = mo > -INFINITY ? ex2_approx(mo - m) : 0.f;
            const float inv_l = 1.f / (l * a_me + lo * a_ot);
            const float w_mine = a_me * inv_l, w_other = a_ot * inv_l;
            // ---- output: this thread's half of the head dimension, from both accumulators ----
            if (!wait_all(&o_full, it & 1)) { ok = false; break; }
            ATTN_T(t6b);
            ATTN_ACC(9, t6a, t6b);
            tc_fence_after();
            // The combined rows go through shared memory: a thread owns a row, so straight from registers a warp's store
            // instruction would touch 32 different lines; staged (16-byte chunks, chunk c of row r at position c ^ (r mod 8)
            // within its 128 bytes) each instruction of the copy-out writes whole rows.
            constexpr int ROWB = HD * 2, CH = HD / 8;          // bytes and 16-byte chunks per output row
#pragma unroll
            for (int ch = 0; ch < HD / 64; ++ch) {
                float a[32], bb[32];
                const int col = hf * (HD / 2) + ch * 32;
                tmem_ld32(lane_base + O_COL + hf * 128 + col, a);
                tmem_ld32(lane_base + O_COL + (hf ^ 1) * 128 + col, bb);
                tmem_ld_wait_regs(a);
                tmem_ld_wait_regs(bb);
#pragma unroll
                for (int g4 = 0; g4 < 4; ++g4) {
                    uint4 ov;
                    __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int e = g4 * 8 + 2 * t;
                        o2[t] = __floats2bfloat162_rn(a[e] * w_mine + bb[e] * w_other, a[e + 1] * w_mine + bb[e + 1] * w_other);
                    }
                    const int cidx = col / 8 + g4;
                    *reinterpret_cast<uint4*>(sO + r * ROWB + ((cidx ^ (r & 7)) << 4)) = ov;
                }
            }
            // the accumulators are read: the next item's first P.V may overwrite them
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&o_empty);
            asm volatile("bar.sync 1, %0;" ::"n"(kAttnSoftmaxThreads) : "memory");      // the 8 softmax warps: the tile is staged
            {
                // softmax warp w copies rows 16 w .. 16 w + 15, 32 / CH rows per instruction.  (The staging buffer is
                // written again only after every warp has passed the next item's exchange barrier, i.e. finished this.)
                const int w8 = warp - 2;
#pragma unroll
                for (int i = 0; i < 16 * CH / 32; ++i) {
                    const int row = w8 * 16 + i * (32 / CH) + lane / CH, cidx = lane % CH;
                    const int q = q_blk * 128 + row;
                    if (q < p.q_cnt) {
                        const uint4 ov = *reinterpret_cast<const uint4*>(sO + row * ROWB + ((cidx ^ (row & 7)) << 4));
                        *reinterpret_cast<uint4*>(p.out + ((size_t)b * p.q_cnt + q) * (size_t)(p.nq * HD) + h * HD + cidx * 8) = ov;
                    }
                }
            }
            ATTN_T(t7);
            ATTN_ACC(5, t6, t7);
        }
        ATTN_T(t_role1);
        ATTN_ACC(7, t_role0, t_role1);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
    if (threadIdx.x == 0 && abort_flag && p.status) atomicExch(p.status, 2);
}

}  // namespace jot
