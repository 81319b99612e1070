// CTA-pair variant of the projection kernel (tcgen05 cta_group::2): two CTAs of a cluster share one
// 256 x 256 output tile.  Each CTA loads its own 128 rows of A and its own half (128 rows) of the W tile,
// the even-ranked CTA issues UMMA 256 x 256 x 16 for both, and each CTA's tensor memory receives its
// 128 rows x 256 columns, which its own epilogue warps drain.  Per CTA and k-block that is 32 KB of
// operands for the same 4.2 MFLOP that cost the one-CTA kernel 48 KB, which is what the shared-memory
// ingest of an SM limits.  Epilogues are those of gemm.cuh (store, SwiGLU, QKV + RoPE, LM-head statistics).
//
// Barriers (same shared-memory offsets in both CTAs):
//   full[s]      leader's only: 1 arrival (leader's expect_tx for both CTAs' bytes) + bytes of both CTAs' loads
//   empty[s]     each CTA's own: arrives through the leader's commit, delivered to both CTAs
//   acc_full[a]  each CTA's own: same mechanism
//   acc_empty[a] leader's only: 8 arrivals = 4 epilogue warps x 2 CTAs (the peer arrives remotely)
#pragma once
#include "gemm.cuh"

namespace jot {

constexpr int kPairStages = 6;
constexpr int kPairStageBytes = 2 * kBM * kBK * 2;                 // A tile + half W tile per CTA
constexpr int kPairDynBytes = kPairStages * kPairStageBytes + 1024;

// Row-block pairs and vocabulary chunks of the pair kernel's LM-head schedule.
__host__ __device__ inline void stats_partition_pair(int R, int n_clusters, int n_vt, int* n_rb, int* n_pr, int* n_ch) {
    const int rb = (R + kBM - 1) / kBM, pr = (rb + 1) / 2;
    int ch = pr > 0 ? n_clusters / pr : 0;
    if (ch > n_vt) ch = n_vt;
    *n_rb = rb;
    *n_pr = pr;
    *n_ch = ch;
}

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
gemm_pair_kernel(const GemmParams p, const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB) {
    constexpr int BN = 256, STAGES = kPairStages;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC = umma_idesc_bf16(256, BN);
    constexpr int HALF_BYTES = kBM * kBK * 2;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)cluster_ctarank();
    const bool leader = rank == 0;
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    const int num_kb = (p.K + kBK - 1) / kBK;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&acc_full[a], 1);
            mbar_init(&acc_empty[a], 8);
        }
        fence_barrier_init();
        fence_proxy_async_smem();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        tmem_alloc_pair(&tmem_base_slot, TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    cluster_sync_all();                       // both CTAs' barriers exist before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    // as in the one-CTA kernel: the LM-head schedule needs a device word of the preceding kernel; the other
    // epilogues let each role wait for itself, the producer after it has requested its first W tiles
    grid_launch_dependents();
    if (is_stats(EPI)) grid_dependency_wait();

    // ---- schedule: pair tiles (two row blocks x one 256-wide column block), identical in every role ----
    const int num_m = (p.M + kBM - 1) / kBM, num_pm = (num_m + 1) / 2;
    constexpr int BN_OUT = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
    const int n_out = (EPI == EPI_SWIGLU) ? p.N / 2 : p.N;
    const int num_n = (n_out + BN_OUT - 1) / BN_OUT;
    int total_tiles = num_pm * num_n;
    int m_blk0 = 0, n_first = 0, chunk = 0;
    bool stats_row_block_valid = false;
    if (is_stats(EPI)) {
        // only the tiles that touch the vocabulary slice [col_lo, col_hi) are visited
        const int stats_hi = p.col_hi > 0 ? p.col_hi : p.N;
        const int tile_lo = p.col_lo / BN, num_nt = (stats_hi + BN - 1) / BN - tile_lo;
        int n_rb, n_pr, n_ch;
        stats_partition_pair(*p.d_R, n_clusters, num_nt, &n_rb, &n_pr, &n_ch);
        chunk = n_pr > 0 ? cluster_id / n_pr : 0;
        total_tiles = 0;
        if (n_pr > 0 && chunk < n_ch) {
            m_blk0 = 2 * (cluster_id % n_pr) + rank;
            stats_row_block_valid = m_blk0 < n_rb;
            n_first = (int)((long long)chunk * num_nt / n_ch);
            total_tiles = (int)((long long)(chunk + 1) * num_nt / n_ch) - n_first;
            n_first += tile_lo;
        }
    }
    auto tile_at = [&](int it, int& m_blk, int& n_blk) -> bool {
        if (is_stats(EPI)) {
            if (it >= total_tiles) return false;
            m_blk = m_blk0;
            n_blk = n_first + it;
            return true;
        }
        const int t = cluster_id + it * n_clusters;
        if (t >= total_tiles) return false;
        m_blk = 2 * (t % num_pm) + rank;          // row-block pairs fastest: neighbours share the W tile
        n_blk = t / num_pm;
        return true;
    };

    if (warp == 0) {
        // ================= TMA producer (both CTAs; the whole warp runs the loop, one lane issues) =================
        const bool elected = elect_one();
        int stage = 0;
        uint32_t phase = 0;
        int m_blk, n_blk;
        bool ok = true;
        // this CTA's half of the W tile: SwiGLU pairs 128 gate rows (leader) with the matching 128 up rows
        auto w_row_of = [&](int nb) {
            return (EPI == EPI_SWIGLU) ? (rank == 0 ? nb * kBM : p.N / 2 + nb * kBM) : nb * BN + rank * kBM;
        };
        // the first tile's first W tiles go out before the wait on the preceding kernel, its A tiles after
        int n_pre = 0;
        if (!is_stats(EPI)) {
            if (tile_at(0, m_blk, n_blk)) {
                n_pre = min(STAGES, num_kb);
                if (elected)
                    for (int i = 0; i < n_pre; ++i) {
                        if (leader) mbar_arrive_expect_tx(&full_bar[i], 2 * kPairStageBytes);
                        tma_load_2d_pair(smem + i * kPairStageBytes + HALF_BYTES, &tmB, mapa_u32(&full_bar[i], 0), i * kBK,
                                         w_row_of(n_blk));
                    }
            }
            __syncwarp();
            grid_dependency_wait();
            if (elected)
                for (int i = 0; i < n_pre; ++i)
                    tma_load_2d_pair(smem + i * kPairStageBytes, &tmA, mapa_u32(&full_bar[i], 0), i * kBK, m_blk * kBM);
            __syncwarp();
        }
        for (int it = 0; ok && tile_at(it, m_blk, n_blk); ++it) {
            const int w_row = w_row_of(n_blk);
            for (int kb = 0; kb < num_kb; ++kb) {
                if (it == 0 && kb < n_pre) {                  // already requested above
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    continue;
                }
                if (!mbar_wait(&empty_bar[stage], phase ^ 1, abortp)) { ok = false; break; }
                uint8_t* sA = smem + stage * kPairStageBytes;
                uint8_t* sB = sA + HALF_BYTES;
                const uint32_t full_leader = mapa_u32(&full_bar[stage], 0);
                if (elected) {
                    if (leader) mbar_arrive_expect_tx(&full_bar[stage], 2 * kPairStageBytes);
                    tma_load_2d_pair(sA, &tmA, full_leader, kb * kBK, m_blk * kBM);
                    tma_load_2d_pair(sB, &tmB, full_leader, kb * kBK, w_row);
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer (leader CTA only; the whole warp runs the loop, one lane issues) ==========
        // One thread issues every MMA of the pair, so the loop is kept to a few instructions per MMA: the operand
        // descriptors of a stage differ from stage 0's only in the 16-byte-granular address field and are
        // advanced by additions (the field never carries: shared-memory addresses stay below 256 KB).
        if (leader) {
            const bool elected = elect_one();
            const uint64_t ad0 = umma_desc_k128(smem_u32(smem));
            const uint64_t bd0 = ad0 + (HALF_BYTES >> 4);
            constexpr uint32_t STAGE_UNITS = kPairStageBytes >> 4;
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
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(&full_bar[stage], phase, abortp)) { ok = false; break; }
                    tc_fence_after();
                    if (elected) {
#pragma unroll
                        for (int k = 0; k < kBK / 16; ++k) umma_bf16_pair(d_tmem, ad + 2 * k, bd + 2 * k, IDESC, accum | k);
                        umma_commit_pair(&empty_bar[stage], 0x3);     // both CTAs may refill this stage
                    }
                    __syncwarp();
                    accum = 1;
                    ad += STAGE_UNITS;
                    bd += STAGE_UNITS;
                    if (++stage == STAGES) { stage = 0; phase ^= 1; ad = ad0; bd = bd0; }
                }
                if (!ok) break;
                if (elected) umma_commit_pair(&acc_full[acc], 0x3);   // both CTAs' accumulators are complete
                __syncwarp();
                if (++acc == 2) { acc = 0; acc_phase ^= 1; }
            }
        }
        __syncwarp();
    } else {
        // ================= epilogue (warps 2..5, both CTAs) =================
        if (!is_stats(EPI)) grid_dependency_wait();
        const int quad = warp & 3;
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
            epilogue_tile<BN, EPI>(p, lane_base + acc * BN, m_blk * kBM + row_in_tile, n_blk, 0, n_out, st);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_u32(&acc_empty[acc], 0));
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
        if (is_stats(EPI) && ok && total_tiles > 0 && stats_row_block_valid) {
            const size_t slot = (size_t)chunk * p.R_pad + m_blk0 * kBM + row_in_tile;
            p.partials[slot] = make_float4(st.m1, __int_as_float(st.i1), st.m2, st.S);
            if (EPI == EPI_STATS_DRAW) p.partials2[slot] = make_float2(st.best, __int_as_float(st.best_i));
        }
    }

    // ---- teardown: nobody leaves while the other CTA may still signal or read across ----
    tc_fence_before();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
    if (threadIdx.x == 0 && abort_flag && p.status) atomicExch(p.status, 3);
}

}  // namespace jot
