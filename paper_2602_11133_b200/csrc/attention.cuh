// Bidirectional (unmasked) grouped-query softmax attention on tcgen05 / tensor memory, fed by TMA.
//
// Persistent CTAs walk over work items (query block of 128 rows, query head, sequence), ordered so that the
// CTAs running side by side share K and V of one KV head in L2.  For one item the keys are visited in blocks
// of 128, twice:
//   pass 1   S = Q K^T per key block -> exact row maximum m
//   pass 2   S again; P = bf16(exp((S - m) / sqrt(hd))) written to shared memory as the A operand of
//            O += P V ; row sum l accumulated in fp32 from the unrounded exponentials
// and finally O / l is written as bf16.  Knowing m before any P is formed means the accumulator in tensor
// memory is never rescaled and P is rounded against the true maximum.
//
//   warp 0 (one lane)  TMA producer: Q per item, K blocks (both passes), V^T blocks (pass 2)
//   warp 1 (one lane)  MMA issuer; S double buffered in tensor memory (S(g+1) overlaps softmax(g)), O double
//                      buffered across items (the output of item i drains while item i+1 accumulates)
//   warps 2..9         softmax: two threads per query row (TMEM lane), each owning 64 of the 128 key columns
//                      of a block and half of the output columns; row max and row sum meet in shared memory
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
    static constexpr int P_BYTES = 2 * 128 * 128;
    static constexpr int DYN_BYTES = Q_BYTES + 2 * K_BYTES + 2 * V_BYTES + P_BYTES + 1024;
};

template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tmQKV, const __grid_constant__ CUtensorMap tmVt) {
    using SM = AttnSmem<HD>;
    constexpr int KB = SM::KB;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC_S = umma_idesc_bf16(128, 128);
    constexpr uint32_t IDESC_O = umma_idesc_bf16(128, HD);
    constexpr uint32_t O_COL = 256;            // S buffers at columns 0 and 128, O buffers at 256 and 384

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + SM::Q_BYTES;          // 2 stages
    uint8_t* sV = sK + 2 * SM::K_BYTES;      // 2 stages
    uint8_t* sP = sV + 2 * SM::V_BYTES;
    __shared__ uint64_t q_full, q_empty, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], s_empty[2], p_full,
        p_empty, o_full[2], o_empty[2], xmax_bar, xsum_bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ float x_max[2][128], x_sum[2][128];

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
            mbar_init(&s_empty[i], 8);
            mbar_init(&o_full[i], 1);
            mbar_init(&o_empty[i], 8);
        }
        mbar_init(&p_full, kAttnSoftmaxThreads);
        mbar_init(&p_empty, 1);
        mbar_init(&xmax_bar, kAttnSoftmaxThreads);
        mbar_init(&xsum_bar, kAttnSoftmaxThreads);
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
            uint32_t gk = 0, gv = 0;     // running counts of K loads (= S products) and V loads (= P.V products)
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
                for (int g = 0; g < 2 * nkb; ++g, ++gk) {
                    const int j = g % nkb, st = gk & 1;
                    if (!mbar_wait(&k_empty[st], ((gk >> 1) & 1) ^ 1, abortp)) { ok = false; break; }
                    mbar_arrive_expect_tx(&k_full[st], SM::K_BYTES);
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb)
                        tma_load_3d(sK + st * SM::K_BYTES + kb * 16384, &tmQKV, &k_full[st], k_col + kb * 64, j * 128, b);
                    if (g >= nkb) {
                        const int vs = gv & 1;
                        if (!mbar_wait(&v_empty[vs], ((gv >> 1) & 1) ^ 1, abortp)) { ok = false; break; }
                        mbar_arrive_expect_tx(&v_full[vs], SM::V_BYTES);
#pragma unroll
                        for (int half = 0; half < 2; ++half)
                            tma_load_2d(sV + vs * SM::V_BYTES + half * (HD * 128), &tmVt, &v_full[vs],
                                        j * 128 + half * 64, vt_row);
                        ++gv;
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t gk = 0, gv = 0;
            int it = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++it) {
                const uint32_t o_tmem = tmem_base + O_COL + (it & 1) * 128;
                auto issue_S = [&](bool last) -> bool {
                    const int st = gk & 1;
                    if (!mbar_wait(&k_full[st], (gk >> 1) & 1, abortp)) return false;
                    if (!mbar_wait(&s_empty[st], ((gk >> 1) & 1) ^ 1, abortp)) return false;
                    tc_fence_after();
                    const uint32_t qa = smem_u32(sQ), ka = smem_u32(sK + st * SM::K_BYTES);
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_bf16(tmem_base + st * 128, umma_desc_k128(qa + kb * 16384 + k * 32),
                                      umma_desc_k128(ka + kb * 16384 + k * 32), IDESC_S, (kb | k) != 0);
                    umma_commit(&k_empty[st]);
                    umma_commit(&s_full[st]);
                    if (last) umma_commit(&q_empty);          // Q may now be overwritten by the next item's
                    ++gk;
                    return true;
                };
                auto issue_PV = [&](int j) -> bool {
                    const int vs = gv & 1;
                    if (!mbar_wait(&v_full[vs], (gv >> 1) & 1, abortp)) return false;
                    if (!mbar_wait(&p_full, gv & 1, abortp)) return false;
                    tc_fence_after();
                    const uint32_t pa = smem_u32(sP), va = smem_u32(sV + vs * SM::V_BYTES);
#pragma unroll
                    for (int half = 0; half < 2; ++half)
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_bf16(o_tmem, umma_desc_k128(pa + half * 16384 + k * 32),
                                      umma_desc_k128(va + half * (HD * 128) + k * 32), IDESC_O, (j | half | k) != 0);
                    umma_commit(&v_empty[vs]);
                    umma_commit(&p_empty);
                    if (j == nkb - 1) umma_commit(&o_full[it & 1]);
                    ++gv;
                    return true;
                };
                ok = mbar_wait(&q_full, it & 1, abortp);
                // this item's O buffer must have been drained by the output step of the item two before
                ok = ok && mbar_wait(&o_empty[it & 1], ((it >> 1) & 1) ^ 1, abortp);
                ok = ok && issue_S(false);
                for (int g = 1; ok && g < 2 * nkb; ++g) {
                    ok = issue_S(g == 2 * nkb - 1);
                    if (ok && g - 1 >= nkb) ok = issue_PV(g - 1 - nkb);
                }
                if (ok) ok = issue_PV(nkb - 1);
            }
        }
    } else {
        // ======== softmax: thread (r, hf) owns row r and key columns [64 hf, 64 hf + 64) of every block ========
        const int quad = warp & 3, hf = (warp - 2) >> 2;
        const int r = quad * 32 + lane;
        const uint32_t lane_base = tmem_base + (uint32_t(quad * 32) << 16);
        const float c = p.scale_log2e;
        uint32_t gk = 0, gv = 0;
        int it = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++it) {
            int q_blk, h, b;
            decode(item, q_blk, h, b);
            // ---- pass 1: row maximum of the raw scores ----
            float m = -INFINITY;
            for (int j = 0; ok && j < nkb; ++j, ++gk) {
                const int st = gk & 1;
                if (!mbar_wait(&s_full[st], (gk >> 1) & 1, abortp)) { ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    float v[32];
                    tmem_ld32(lane_base + st * 128 + hf * 64 + ch * 32, v);
                    tmem_ld_wait();
                    const int key0 = j * 128 + hf * 64 + ch * 32;
#pragma unroll
                    for (int t = 0; t < 32; ++t) m = (key0 + t < L) ? fmaxf(m, v[t]) : m;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_empty[st]);
            }
            if (!ok) break;
            // the two halves of a row meet (bounded wait, like every other wait in this kernel)
            x_max[hf][r] = m;
            mbar_arrive(&xmax_bar);
            if (!mbar_wait(&xmax_bar, it & 1, abortp)) { ok = false; break; }
            m = fmaxf(m, x_max[hf ^ 1][r]);
            // ---- pass 2: probabilities, P to shared memory, row sum ----
            const float mc = m * c;
            float l = 0.f;
            for (int j = 0; ok && j < nkb; ++j, ++gk, ++gv) {
                const int st = gk & 1;
                if (!mbar_wait(&s_full[st], (gk >> 1) & 1, abortp)) { ok = false; break; }
                tc_fence_after();
                uint32_t packed[32];
#pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    float v[32];
                    tmem_ld32(lane_base + st * 128 + hf * 64 + ch * 32, v);
                    tmem_ld_wait();
                    const int key0 = j * 128 + hf * 64 + ch * 32;
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        float e0 = (key0 + 2 * t < L) ? ex2_approx(fmaf(v[2 * t], c, -mc)) : 0.f;
                        float e1 = (key0 + 2 * t + 1 < L) ? ex2_approx(fmaf(v[2 * t + 1], c, -mc)) : 0.f;
                        l += e0 + e1;
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(e0, e1);
                        packed[ch * 16 + t] = *reinterpret_cast<uint32_t*>(&h2);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_empty[st]);
                // P buffer free once the previous P.V has retired
                if (!mbar_wait(&p_empty, (gv & 1) ^ 1, abortp)) { ok = false; break; }
                // this thread's 64 keys = sub-tile hf of P, row r: 8 chunks of 16 bytes, 128-byte swizzle
#pragma unroll
                for (int cc = 0; cc < 8; ++cc) {
                    uint8_t* dst = sP + hf * 16384 + r * 128 + ((cc ^ (r & 7)) << 4);
                    *reinterpret_cast<uint4*>(dst) =
                        make_uint4(packed[cc * 4], packed[cc * 4 + 1], packed[cc * 4 + 2], packed[cc * 4 + 3]);
                }
                fence_proxy_async_smem();
                mbar_arrive(&p_full);
            }
            if (!ok) break;
            x_sum[hf][r] = l;
            mbar_arrive(&xsum_bar);
            if (!mbar_wait(&xsum_bar, it & 1, abortp)) { ok = false; break; }
            l += x_sum[hf ^ 1][r];
            // ---- output: this thread's half of the head dimension ----
            if (!mbar_wait(&o_full[it & 1], (it >> 1) & 1, abortp)) { ok = false; break; }
            tc_fence_after();
            const int q = q_blk * 128 + r;
            const float inv_l = 1.f / l;
#pragma unroll
            for (int ch = 0; ch < HD / 64; ++ch) {
                float v[32];
                const int col = hf * (HD / 2) + ch * 32;
                tmem_ld32(lane_base + O_COL + (it & 1) * 128 + col, v);
                tmem_ld_wait();
                if (q < p.q_cnt) {
                    __nv_bfloat16* dst = p.out + ((size_t)b * p.q_cnt + q) * (size_t)(p.nq * HD) + h * HD + col;
#pragma unroll
                    for (int g4 = 0; g4 < 4; ++g4) {
                        uint4 ov;
                        __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
                        for (int t = 0; t < 4; ++t)
                            o2[t] = __floats2bfloat162_rn(v[g4 * 8 + 2 * t] * inv_l, v[g4 * 8 + 2 * t + 1] * inv_l);
                        *reinterpret_cast<uint4*>(dst + g4 * 8) = ov;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&o_empty[it & 1]);
        }
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
