// Acceptance / freeze update of one denoising step: one CTA per sequence.
// Section 4.1 of the paper: confidence ratio (Eq. 4), spatial weight over a window of radius D (Eq. 5),
// softening factor (Eq. 6), adaptive threshold (Eq. 7), early-exit test (Eq. 8); then the transfer
// schedule (k highest max-probability candidates), the logical OR of both masks, and the write of
// the argmax token into every chosen position (Algorithm 1).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "pdl.cuh"

namespace jot {

constexpr int kAcceptThreads = 256;
constexpr int kMaxD = 32;

struct AcceptParamsDev {     // mirrors jot_params
    float tau_max, tau_min, gamma;
    int32_t D;
    float eps;
    int32_t schedule_after_exit;
    int32_t gate;                // 0: ratio r >= tau (Eq. 8); 1: fixed probability gate p1 >= prob_threshold;
    float prob_threshold;        // 2: global early commit, mean top-2 logit gap of the candidates >= gap_threshold
    float gap_threshold;
    int32_t schedule;            // 0: fixed per-block table; 1: ceil(still masked / steps the block has left)
};

// Per-sequence loop state used by the generate loop (device resident).
struct SeqState {
    int32_t blk;          // current semi-autoregressive block
    int32_t s;            // step inside the block
    int32_t steps_used;   // denoising steps this sequence has run
    int32_t n_masked;     // candidates still masked in the current block after the last update
};

struct AcceptArgs {
    AcceptParamsDev uniform;         // used when params == nullptr
    const AcceptParamsDev* params;   // device: 1 or B entries (nullable)
    int per_seq_params;
    int32_t mask_id;
    int32_t* tokens;                 // [B, L], updated in place
    int B, L;
    int blk_lo, blk_hi, k_transfer;  // used when state == nullptr
    const float* top1;
    const float* top2;
    const float* sumexp;
    const int32_t* argmax;
    int32_t* n_masked;               // [B] nullable
    uint8_t* exit_reason;            // [B, L] nullable
    int16_t* exit_step;              // [B, L] nullable
    int step_index;
    // generate mode: block pointer / step per sequence, schedule table from (block_len, steps_per_block)
    SeqState* state;                 // [B] nullable
    int P, block_len, n_blocks, steps_per_block;
    int32_t* n_unfinished;           // device counter: += 1 per sequence that still has work (nullable)
    int lockstep;                    // generate mode under a block-wise KV cache: every sequence works on the block
                                     // [blk_lo, blk_hi) with k_transfer; the host moves all of them on together
    int lockstep_s;                  // ... and this is the block's step index (the fractional schedule needs it)
    // generate mode, optional trace (Appendix "Confidence Dynamics"): row = the sequence's own 0-based step
    float* mean_ratio;               // [steps, B]: mean of r over the step's candidates
    int32_t* n_candidates;           // [steps, B]
};

// Per-sequence parameter sets handed over as kernel arguments (the single-step entry point has no device
// memory of its own to put them in): at most this many sequences per launch.
constexpr int kAcceptInlineParams = 64;
struct AcceptParamsInline {
    AcceptParamsDev p[kAcceptInlineParams];
};
struct AcceptParamsNone {};

template <bool INLINE> struct AcceptInlineArg { using type = AcceptParamsNone; };
template <> struct AcceptInlineArg<true> { using type = AcceptParamsInline; };

__device__ __forceinline__ AcceptParamsDev accept_pick_params(const AcceptArgs& a, const AcceptParamsInline& inl, int b) {
    return inl.p[b];
}
__device__ __forceinline__ AcceptParamsDev accept_pick_params(const AcceptArgs& a, const AcceptParamsNone&, int b) {
    return a.params ? a.params[a.per_seq_params ? b : 0] : a.uniform;
}

// Dynamic shared memory: resolved bitmap words, candidate list, candidate sum-exp, candidate flags.
template <bool INLINE>
__global__ void __launch_bounds__(kAcceptThreads)
accept_freeze_kernel(const AcceptArgs a, const __grid_constant__ typename AcceptInlineArg<INLINE>::type inl) {
    extern __shared__ uint32_t sh[];
    grid_launch_dependents();
    grid_dependency_wait();
    const int L = a.L, b = blockIdx.x, tid = threadIdx.x;
    const int n_words = (L + 31) / 32;
    uint32_t* res_bits = sh;                                   // [n_words + 2] resolved bitmap (padded)
    int* cand = reinterpret_cast<int*>(sh + n_words + 2);     // [L] candidate positions, ascending
    float* cand_S = reinterpret_cast<float*>(cand + L);       // [L] their sum-exp (p1 = 1/S)
    uint8_t* cand_flag = reinterpret_cast<uint8_t*>(cand_S + L);   // [L] bit0 exit, bit1 schedule
    __shared__ float gpow[kMaxD + 1];
    __shared__ int n_cand_sh, warp_counts[kAcceptThreads / 32], n_final_sh;
    __shared__ float inv_wmax;
    __shared__ float ratio_sums[kAcceptThreads / 32], gap_sums[kAcceptThreads / 32];

    const AcceptParamsDev prm = accept_pick_params(a, inl, b);
    int32_t* x = a.tokens + (size_t)b * L;

    int lo = a.blk_lo, hi = a.blk_hi, k = a.k_transfer;
    SeqState st = {0, 0, 0, 0};
    if (a.state) st = a.state[b];
    if (a.state && !a.lockstep) {
        if (st.blk >= a.n_blocks) return;                      // finished sequence idles (uniform exit)
        lo = a.P + st.blk * a.block_len;
        hi = lo + a.block_len;
        int base = a.block_len / a.steps_per_block, rem = a.block_len % a.steps_per_block;
        k = base + (st.s < rem ? 1 : 0);
    }

    if (tid == 0) {
        // gamma^d by repeated multiplication, and w_max = 2 * sum_{d=1..D} gamma^d  (Eq. 6)
        float g = 1.f, sum = 0.f;
        gpow[0] = 0.f;
        for (int d = 1; d <= prm.D; ++d) {
            g *= prm.gamma;
            gpow[d] = g;
            sum += g;
        }
        inv_wmax = 1.f / (2.f * sum);
        n_cand_sh = 0;
        n_final_sh = 0;
    }
    // resolved bitmap: bit i set iff x_i != mask_id (prompt tokens count as resolved)
    for (int w = tid; w < n_words + 2; w += blockDim.x) res_bits[w] = 0;
    __syncthreads();
    for (int base = 0; base < L; base += blockDim.x) {
        int i = base + tid;
        bool r = (i < L) && (x[i] != a.mask_id);
        uint32_t bal = __ballot_sync(0xffffffffu, r);
        if ((tid & 31) == 0 && (i >> 5) < n_words) res_bits[i >> 5] = bal;
    }
    __syncthreads();

    // candidate list in ascending position order (block-wide compaction, chunk by chunk)
    for (int base = lo; base < hi; base += blockDim.x) {
        int i = base + tid;
        bool c = (i < hi) && !((res_bits[i >> 5] >> (i & 31)) & 1u);
        uint32_t bal = __ballot_sync(0xffffffffu, c);
        int wid = tid >> 5, ln = tid & 31;
        if (ln == 0) warp_counts[wid] = __popc(bal);
        __syncthreads();
        int off = n_cand_sh;
        for (int w = 0; w < wid; ++w) off += warp_counts[w];
        if (c) cand[off + __popc(bal & ((1u << ln) - 1u))] = i;
        __syncthreads();
        if (tid == 0) {
            int t = 0;
            for (int w = 0; w < kAcceptThreads / 32; ++w) t += warp_counts[w];
            n_cand_sh += t;
        }
        __syncthreads();
    }
    const int n_cand = n_cand_sh;
    if (a.state && prm.schedule == 1) {
        // adaptive schedule: the share of what is still masked that keeps the block on pace to end with its last step
        const int steps_left = max(1, a.steps_per_block - (a.lockstep ? a.lockstep_s : st.s));
        k = (n_cand + steps_left - 1) / steps_left;
    }

    // per candidate: ratio, threshold, early-exit decision
    float r_sum = 0.f, gap_sum = 0.f;
    for (int c = tid; c < n_cand; c += blockDim.x) {
        const int i = cand[c];
        const size_t gi = (size_t)b * L + i;
        const float m1 = a.top1[gi], m2 = a.top2[gi], S = a.sumexp[gi];
        // Eq. 4 with p1 = 1/S, p2 = exp(m2 - m1)/S:  r = 1 / (exp(m2 - m1) + eps * S)
        const float r = 1.f / (expf(m2 - m1) + prm.eps * S);
        // Eq. 5: resolved neighbours at distance 1..D on both sides, read from the bitmap
        float w = 0.f;
        for (int d = 1; d <= prm.D; ++d) {
            int jl = i - d, jr = i + d;
            if (jl >= 0 && ((res_bits[jl >> 5] >> (jl & 31)) & 1u)) w += gpow[d];
            if (jr < L && ((res_bits[jr >> 5] >> (jr & 31)) & 1u)) w += gpow[d];
        }
        const float phi = fminf(1.f, w * inv_wmax);                        // Eq. 6
        const float tau = prm.tau_max - (prm.tau_max - prm.tau_min) * phi; // Eq. 7
        cand_S[c] = S;
        r_sum += r;
        gap_sum += m1 - m2;
        // Eq. 8; or the fixed probability gate the paper contrasts it with (p1 = 1/S, no spatial modulation)
        // (the global early-commit gate decides for all candidates together, after the sum below)
        const bool exit_now = prm.gate == 1 ? (1.f / S >= prm.prob_threshold) : (prm.gate == 2 ? false : r >= tau);
        cand_flag[c] = exit_now ? 1 : 0;
    }
    if (prm.gate == 2) {                                       // fixed-order tree: the same sum on every run
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) gap_sum += __shfl_xor_sync(0xffffffffu, gap_sum, o);
        if ((tid & 31) == 0) gap_sums[tid >> 5] = gap_sum;
    }
    if (a.mean_ratio) {                                        // fixed-order tree: the same sum on every run
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) r_sum += __shfl_xor_sync(0xffffffffu, r_sum, o);
        if ((tid & 31) == 0) ratio_sums[tid >> 5] = r_sum;
    }
    __syncthreads();
    if (prm.gate == 2 && n_cand > 0) {
        // global early commit: every candidate exits when the mean top-2 logit gap clears the threshold
        float t = 0.f;
        for (int w = 0; w < kAcceptThreads / 32; ++w) t += gap_sums[w];
        if (t / (float)n_cand >= prm.gap_threshold)
            for (int c = tid; c < n_cand; c += blockDim.x) cand_flag[c] = 1;
    }
    if (prm.gate == 2) __syncthreads();                        // the schedule below may read other threads' flags

    // transfer schedule: the k candidates with the largest p1 = 1/S, i.e. the smallest S; equal S
    // resolves to the lower position.  Rank by counting (candidate lists are short).
    const int k_eff = min(k, n_cand);
    if (k_eff > 0) {
        for (int c = tid; c < n_cand; c += blockDim.x) {
            const bool skip_exited = prm.schedule_after_exit != 0;
            if (skip_exited && (cand_flag[c] & 1)) continue;
            const float Sc = cand_S[c];
            int rank = 0;
            for (int o = 0; o < n_cand; ++o) {
                if (skip_exited && (cand_flag[o] & 1)) continue;
                const float So = cand_S[o];
                rank += (So < Sc) || (So == Sc && o < c);
            }
            if (rank < k_eff) cand_flag[c] |= 2;
        }
    }
    __syncthreads();

    // freeze: chosen candidates receive their argmax; everything else is left untouched
    int my_final = 0;
    for (int c = tid; c < n_cand; c += blockDim.x) {
        const uint8_t f = cand_flag[c];
        if (f) {
            const int i = cand[c];
            const size_t gi = (size_t)b * L + i;
            x[i] = a.argmax[gi];
            if (a.exit_reason) a.exit_reason[gi] = f;
            if (a.exit_step) a.exit_step[gi] = (int16_t)(a.state ? st.steps_used + 1 : a.step_index);
            ++my_final;
        }
    }
    if (my_final) atomicAdd(&n_final_sh, my_final);
    __syncthreads();
    if (tid == 0) {
        const int left = n_cand - n_final_sh;
        if (a.n_masked) a.n_masked[b] = left;
        if (a.state) {
            if (n_cand > 0 && a.mean_ratio) {
                float t = 0.f;
                for (int w = 0; w < kAcceptThreads / 32; ++w) t += ratio_sums[w];
                a.mean_ratio[(size_t)st.steps_used * a.B + b] = t / (float)n_cand;
            }
            if (n_cand > 0 && a.n_candidates) a.n_candidates[(size_t)st.steps_used * a.B + b] = n_cand;
            if (n_cand > 0) st.steps_used += 1;
            st.n_masked = left;
            if (a.lockstep) {                                  // the host advances the block for everyone
                a.state[b] = st;
                if (a.n_unfinished && left > 0) atomicAdd(a.n_unfinished, 1);
            } else {
                if (left == 0) { st.blk += 1; st.s = 0; } else { st.s += 1; }
                a.state[b] = st;
                if (a.n_unfinished && st.blk < a.n_blocks) atomicAdd(a.n_unfinished, 1);
            }
        }
    }
}

inline size_t accept_smem_bytes(int L) {
    return (size_t)((L + 31) / 32 + 2) * 4 + (size_t)L * 4 + (size_t)L * 4 + (size_t)((L + 3) / 4) * 4 + 16;
}

}  // namespace jot
