// Bidirectional (unmasked) grouped-query softmax attention on tcgen05 / tensor memory, fed by TMA.
//
// One CTA per (query block of 128 rows, query head, sequence).  Keys are visited in blocks of 128, twice:
//   pass 1   S = Q K^T per key block -> exact row maximum m
//   pass 2   S again; P = bf16(exp((S - m) / sqrt(hd))) written to shared memory as the A operand of
//            O += P V ; row sum l accumulated in fp32 from the unrounded exponentials
// and finally O / l is written as bf16.  Knowing m before any P is formed means the accumulator in
// tensor memory is never rescaled and P is rounded against the true maximum.
//
//   warp 0 (one lane)  TMA producer: Q once, K blocks (both passes), V^T blocks (pass 2)
//   warp 1 (one lane)  MMA issuer; S is double buffered in tensor memory so S(g+1) overlaps softmax(g)
//   warps 2..5         softmax: thread r owns query row r (TMEM lane r)
//
// Layouts: qkv [B*L, (nq + 2 nkv) * hd] after RoPE (3-D tensor map (col, position, sequence) so that a
// block never reads across a sequence boundary: out-of-range positions read as zero); V transposed
// vt [B * nkv * hd, Lp] with keys contiguous, so that both products take K-major operands.
#pragma once
#include "pdl.cuh"
#include "ptx.cuh"

namespace jot {

constexpr int kAttnThreads = 192;

struct AttnParams {
    int L, nq, nkv;
    float scale_log2e;            // log2(e) / sqrt(hd)
    __nv_bfloat16* out;           // [B*L, nq*hd]
    int32_t* status;
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
    constexpr uint32_t O_COL = 256;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + SM::Q_BYTES;          // 2 stages
    uint8_t* sV = sK + 2 * SM::K_BYTES;      // 2 stages
    uint8_t* sP = sV + 2 * SM::V_BYTES;
    __shared__ uint64_t q_full, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], s_empty[2], p_full, p_empty,
        o_full;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q_blk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (p.nq / p.nkv);
    const int L = p.L;
    const int nkb = (L + 127) / 128;
    const int q_col = h * HD, k_col = (p.nq + kvh) * HD;
    const int vt_row = (b * p.nkv + kvh) * HD;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&q_full, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&k_full[i], 1);
            mbar_init(&k_empty[i], 1);
            mbar_init(&v_full[i], 1);
            mbar_init(&v_empty[i], 1);
            mbar_init(&s_full[i], 1);
            mbar_init(&s_empty[i], 4);
        }
        mbar_init(&p_full, 128);
        mbar_init(&p_empty, 1);
        mbar_init(&o_full, 1);
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

    if (warp == 0) {
        if (lane == 0) {
            mbar_arrive_expect_tx(&q_full, SM::Q_BYTES);
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
                tma_load_3d(sQ + kb * 16384, &tmQKV, &q_full, q_col + kb * 64, q_blk * 128, b);
            for (int g = 0; g < 2 * nkb; ++g) {
                const int j = g % nkb, st = g & 1;
                if (!mbar_wait(&k_empty[st], ((g >> 1) & 1) ^ 1, abortp)) break;
                mbar_arrive_expect_tx(&k_full[st], SM::K_BYTES);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
                    tma_load_3d(sK + st * SM::K_BYTES + kb * 16384, &tmQKV, &k_full[st], k_col + kb * 64, j * 128, b);
                if (g >= nkb) {
                    const int vs = j & 1;
                    if (!mbar_wait(&v_empty[vs], ((j >> 1) & 1) ^ 1, abortp)) break;
                    mbar_arrive_expect_tx(&v_full[vs], SM::V_BYTES);
#pragma unroll
                    for (int half = 0; half < 2; ++half)
                        tma_load_2d(sV + vs * SM::V_BYTES + half * (HD * 128), &tmVt, &v_full[vs], j * 128 + half * 64,
                                    vt_row);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = mbar_wait(&q_full, 0, abortp);
            auto issue_S = [&](int g) -> bool {
                const int st = g & 1;
                if (!mbar_wait(&k_full[st], (g >> 1) & 1, abortp)) return false;
                if (!mbar_wait(&s_empty[st], ((g >> 1) & 1) ^ 1, abortp)) return false;
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
                return true;
            };
            auto issue_PV = [&](int j) -> bool {
                const int vs = j & 1;
                if (!mbar_wait(&v_full[vs], (j >> 1) & 1, abortp)) return false;
                if (!mbar_wait(&p_full, j & 1, abortp)) return false;
                tc_fence_after();
                const uint32_t pa = smem_u32(sP), va = smem_u32(sV + vs * SM::V_BYTES);
#pragma unroll
                for (int half = 0; half < 2; ++half)
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_bf16(tmem_base + O_COL, umma_desc_k128(pa + half * 16384 + k * 32),
                                  umma_desc_k128(va + half * (HD * 128) + k * 32), IDESC_O, (j | half | k) != 0);
                umma_commit(&v_empty[vs]);
                umma_commit(&p_empty);
                if (j == nkb - 1) umma_commit(&o_full);
                return true;
            };
            ok = ok && issue_S(0);
            for (int g = 1; ok && g < 2 * nkb; ++g) {
                ok = issue_S(g);
                if (ok && g - 1 >= nkb) ok = issue_PV(g - 1 - nkb);
            }
            if (ok) issue_PV(nkb - 1);
        }
    } else {
        const int quad = warp & 3;
        const int r = quad * 32 + lane;                            // query row inside the block
        const uint32_t lane_base = tmem_base + (uint32_t(quad * 32) << 16);
        const float c = p.scale_log2e;
        float m = -INFINITY;
        bool ok = true;
        // ---- pass 1: row maximum of the raw scores ----
        for (int g = 0; ok && g < nkb; ++g) {
            const int st = g & 1;
            if (!mbar_wait(&s_full[st], (g >> 1) & 1, abortp)) { ok = false; break; }
            tc_fence_after();
#pragma unroll 1
            for (int ch = 0; ch < 4; ++ch) {
                float v[32];
                tmem_ld32(lane_base + st * 128 + ch * 32, v);
                tmem_ld_wait();
                const int key0 = g * 128 + ch * 32;
#pragma unroll
                for (int j = 0; j < 32; ++j) m = (key0 + j < L) ? fmaxf(m, v[j]) : m;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_empty[st]);
        }
        // ---- pass 2: probabilities, P to shared memory, row sum ----
        const float mc = m * c;
        float l = 0.f;
        for (int j = 0; ok && j < nkb; ++j) {
            const int g = nkb + j, st = g & 1;
            if (!mbar_wait(&s_full[st], (g >> 1) & 1, abortp)) { ok = false; break; }
            tc_fence_after();
            uint32_t packed[64];
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                float v[32];
                tmem_ld32(lane_base + st * 128 + ch * 32, v);
                tmem_ld_wait();
                const int key0 = j * 128 + ch * 32;
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
            if (!mbar_wait(&p_empty, (j & 1) ^ 1, abortp)) { ok = false; break; }
            // row r of P: 16 chunks of 16 bytes, 128-byte swizzle (chunk index XOR row mod 8)
#pragma unroll
            for (int cc = 0; cc < 16; ++cc) {
                uint8_t* dst = sP + (cc >> 3) * 16384 + r * 128 + (((cc & 7) ^ (r & 7)) << 4);
                *reinterpret_cast<uint4*>(dst) =
                    make_uint4(packed[cc * 4], packed[cc * 4 + 1], packed[cc * 4 + 2], packed[cc * 4 + 3]);
            }
            fence_proxy_async_smem();
            mbar_arrive(&p_full);
        }
        // ---- output ----
        if (ok && mbar_wait(&o_full, 0, abortp)) {
            tc_fence_after();
            const int q = q_blk * 128 + r;
            const float inv_l = 1.f / l;
#pragma unroll 1
            for (int ch = 0; ch < HD / 32; ++ch) {
                float v[32];
                tmem_ld32(lane_base + O_COL + ch * 32, v);
                tmem_ld_wait();
                if (q < L) {
                    __nv_bfloat16* dst = p.out + ((size_t)b * L + q) * (size_t)(p.nq * HD) + h * HD + ch * 32;
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
