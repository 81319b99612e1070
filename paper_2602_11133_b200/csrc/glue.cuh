// Bandwidth-bound pieces of the denoising step: embedding gather, RMSNorm (plain and with active-row
// compaction), split-K tail fused with the next norm, active-row list, merge of the LM-head partial
// statistics, canvas initialisation.  All bf16 activations, fp32 arithmetic, 16-byte accesses.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "accept.cuh"

namespace jot {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Block-wide sum for blockDim.x <= 1024 (result valid in every thread).
__device__ __forceinline__ float block_sum(float v, float* scratch /* >= 33 floats */) {
    v = warp_sum(v);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
    if (l == 0) scratch[w] = v;
    __syncthreads();
    if (w == 0) {
        float t = (l < nw) ? scratch[l] : 0.f;
        t = warp_sum(t);
        if (l == 0) scratch[32] = t;
    }
    __syncthreads();
    float r = scratch[32];
    __syncthreads();
    return r;
}

// h[row, :] = E[token of that row, :]     one CTA per row, 16-byte copies (d multiple of 8).
// The launch covers rows_per_seq consecutive canvas positions of every sequence, starting at pos0 (the whole
// canvas: L, 0): row r is (slot, position) = (r / rows_per_seq, pos0 + r % rows_per_seq).
// With seq_map the slots are those of a compacted batch: slot b' reads tokens[seq_map[b'], position].
// A token id outside [0, vocab) is embedded as token 0 and reported through the status word: no read leaves E.
constexpr int32_t kStatusBadToken = 5;
__global__ void embed_kernel(const int32_t* __restrict__ tokens, const __nv_bfloat16* __restrict__ E,
                             __nv_bfloat16* __restrict__ h, int d, int L, const int32_t* __restrict__ seq_map,
                             int rows_per_seq, int pos0, int vocab, int32_t* status) {
    grid_launch_dependents();
    grid_dependency_wait();
    const int row = blockIdx.x;
    int b = row / rows_per_seq;
    if (seq_map) {
        b = seq_map[b];                                 // unused slots (-1) compute on sequence 0; nobody reads them
        b = b < 0 ? 0 : b;
    }
    const int src_row = b * L + pos0 + row % rows_per_seq;
    int tok = tokens[src_row];
    if ((unsigned)tok >= (unsigned)vocab) {
        if (threadIdx.x == 0 && status) atomicCAS(status, 0, kStatusBadToken);   // an expired wait, if any, stays on record
        tok = 0;
    }
    const uint4* src = reinterpret_cast<const uint4*>(E + (size_t)tok * d);
    uint4* dst = reinterpret_cast<uint4*>(h + (size_t)row * d);
    for (int i = threadIdx.x; i < d / 8; i += blockDim.x) dst[i] = src[i];
}

// out[r, :] = bf16( x[src_row, :] * rsqrt(mean(x^2) + eps) * gain ),  src_row = rows ? rows[r] : r.
// With `rows`, only r < *d_R is processed (final norm + compaction of the active rows).
// One CTA per output row; d multiple of 8 and d/8 <= 8 * blockDim.x.
__global__ void rmsnorm_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ gain,
                               __nv_bfloat16* __restrict__ out, int d, float eps, const int32_t* __restrict__ rows,
                               const int32_t* __restrict__ d_R) {
    grid_launch_dependents();
    grid_dependency_wait();
    __shared__ float scratch[33];
    const int r = blockIdx.x;
    int src = r;
    if (rows) {
        if (r >= *d_R) return;
        src = rows[r];
    }
    const uint4* xin = reinterpret_cast<const uint4*>(x + (size_t)src * d);
    const int nvec = d / 8;
    constexpr int MAXV = 8;
    uint4 buf[MAXV];
    float ss = 0.f;
#pragma unroll
    for (int t = 0; t < MAXV; ++t) {
        int i = threadIdx.x + t * blockDim.x;
        if (i < nvec) {
            buf[t] = xin[i];
            const __nv_bfloat162* b2 = reinterpret_cast<const __nv_bfloat162*>(&buf[t]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float2 f = __bfloat1622float2(b2[j]);
                ss += f.x * f.x + f.y * f.y;
            }
        }
    }
    ss = block_sum(ss, scratch);
    const float inv = rsqrtf(ss / (float)d + eps);
    const uint4* g4 = reinterpret_cast<const uint4*>(gain);
    uint4* o4 = reinterpret_cast<uint4*>(out + (size_t)r * d);
#pragma unroll
    for (int t = 0; t < MAXV; ++t) {
        int i = threadIdx.x + t * blockDim.x;
        if (i < nvec) {
            uint4 gv = g4[i], ov;
            const __nv_bfloat162* b2 = reinterpret_cast<const __nv_bfloat162*>(&buf[t]);
            const __nv_bfloat162* g2 = reinterpret_cast<const __nv_bfloat162*>(&gv);
            __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float2 f = __bfloat1622float2(b2[j]), g = __bfloat1622float2(g2[j]);
                o2[j] = __floats2bfloat162_rn(f.x * inv * g.x, f.y * inv * g.y);
            }
            o4[i] = ov;
        }
    }
}

// Split-K tail fused with the next RMSNorm: one CTA per row, one (at most two) 8-element vectors per thread,
// every load of a thread issued before the first use so that a row costs one round trip to L2.
//   h[row, :]   = bf16( sum over K ranges of partial + residual )          (the projection's output)
//   out[row, :] = bf16( h * rsqrt(mean(h^2) + eps) * gain )                (h as rounded, like rmsnorm_kernel)
// N multiple of 8, N/8 <= 2 * blockDim.x (at most 512 threads), split <= 4.
__global__ void __launch_bounds__(512) splitk_reduce_norm_kernel(const float* __restrict__ partial, int split,
                                                                  const __nv_bfloat16* residual, __nv_bfloat16* C, int M,
                                                                  int N, const __nv_bfloat16* __restrict__ gain,
                                                                  __nv_bfloat16* __restrict__ out, float eps) {
    grid_launch_dependents();
    __shared__ float scratch[33];
    const int row = blockIdx.x, nvec = N / 8;
    const size_t total = (size_t)M * N, base = (size_t)row * N;
    constexpr int MAXV = 2, MAXS = 4;
    float4 pa[MAXV][MAXS][2];
    uint4 rv[MAXV], gv[MAXV];
    // The gain is a weight, nobody's output: it is requested before the wait on the preceding kernel.  (The
    // residual is not: with programmatic launches the kernel before the preceding one may still be writing it.)
#pragma unroll
    for (int t = 0; t < MAXV; ++t) {
        const int i = threadIdx.x + t * blockDim.x;
        if (i < nvec) gv[t] = *reinterpret_cast<const uint4*>(gain + i * 8);
    }
    grid_dependency_wait();
#pragma unroll
    for (int t = 0; t < MAXV; ++t) {
        const int i = threadIdx.x + t * blockDim.x;
        if (i < nvec) {
            rv[t] = residual ? *reinterpret_cast<const uint4*>(residual + base + i * 8) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int s = 0; s < MAXS; ++s)
                if (s < split) {
                    pa[t][s][0] = *reinterpret_cast<const float4*>(partial + s * total + base + i * 8);
                    pa[t][s][1] = *reinterpret_cast<const float4*>(partial + s * total + base + i * 8 + 4);
                }
        }
    }
    uint4 hbuf[MAXV];
    float ss = 0.f;
#pragma unroll
    for (int t = 0; t < MAXV; ++t) {
        const int i = threadIdx.x + t * blockDim.x;
        if (i < nvec) {
            float x[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) x[j] = 0.f;
#pragma unroll
            for (int s = 0; s < MAXS; ++s)
                if (s < split) {
                    const float4 a = pa[t][s][0], b = pa[t][s][1];
                    x[0] += a.x; x[1] += a.y; x[2] += a.z; x[3] += a.w;
                    x[4] += b.x; x[5] += b.y; x[6] += b.z; x[7] += b.w;
                }
            const __nv_bfloat162* r2 = reinterpret_cast<const __nv_bfloat162*>(&rv[t]);
            __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&hbuf[t]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 f = __bfloat1622float2(r2[j]);        // zero when there is no residual
                o2[j] = __floats2bfloat162_rn(x[2 * j] + f.x, x[2 * j + 1] + f.y);
                const float2 hr = __bfloat1622float2(o2[j]);
                ss += hr.x * hr.x + hr.y * hr.y;
            }
            *reinterpret_cast<uint4*>(C + base + i * 8) = hbuf[t];
        }
    }
    ss = block_sum(ss, scratch);
    const float inv = rsqrtf(ss / (float)N + eps);
#pragma unroll
    for (int t = 0; t < MAXV; ++t) {
        const int i = threadIdx.x + t * blockDim.x;
        if (i < nvec) {
            uint4 ov;
            const __nv_bfloat162* b2 = reinterpret_cast<const __nv_bfloat162*>(&hbuf[t]);
            const __nv_bfloat162* g2 = reinterpret_cast<const __nv_bfloat162*>(&gv[t]);
            __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 f = __bfloat1622float2(b2[j]), g = __bfloat1622float2(g2[j]);
                o2[j] = __floats2bfloat162_rn(f.x * inv * g.x, f.y * inv * g.y);
            }
            *reinterpret_cast<uint4*>(out + base + i * 8) = ov;
        }
    }
}

// Active rows of the step: every position of [lo_b, hi_b) that holds mask_id, in (b, i) order.
// Single CTA.  rows_out[r] = b*L + i (index into the caller's [B, L] arrays); rows[r] = the same row's index
// in the forward pass's activation matrix, which differs when finished sequences were compacted away
// (seq_map: compact slot -> sequence; n_seq slots) or when the pass covered only positions pos0 ..
// pos0 + rows_per_seq - 1 of every sequence (the whole canvas: rows_per_seq = L, pos0 = 0).  *d_R = count.  With `state`, each sequence uses its
// own block and finished sequences contribute nothing.
__global__ void __launch_bounds__(1024) build_rows_kernel(const int32_t* __restrict__ tokens, int B, int L,
                                                          int32_t mask_id, int blk_lo, int blk_hi,
                                                          const SeqState* __restrict__ state, int P, int block_len,
                                                          int n_blocks, const int32_t* __restrict__ seq_map,
                                                          int32_t* __restrict__ rows, int32_t* __restrict__ rows_out,
                                                          int32_t* __restrict__ d_R, int rows_per_seq, int pos0) {
    grid_launch_dependents();
    grid_dependency_wait();
    __shared__ int warp_counts[32];
    __shared__ int total;
    const int tid = threadIdx.x, wid = tid >> 5, ln = tid & 31;
    if (tid == 0) total = 0;
    __syncthreads();
    for (int slot = 0; slot < B; ++slot) {
        const int b = seq_map ? seq_map[slot] : slot;
        if (b < 0) continue;                                // unused slot of a compacted batch
        int lo = blk_lo, hi = blk_hi;
        if (state) {
            const int blk = state[b].blk;
            if (blk >= n_blocks) continue;
            lo = P + blk * block_len;
            hi = lo + block_len;
        }
        for (int base = lo; base < hi; base += blockDim.x) {
            const int i = base + tid;
            const bool c = (i < hi) && tokens[(size_t)b * L + i] == mask_id;
            const uint32_t bal = __ballot_sync(0xffffffffu, c);
            if (ln == 0) warp_counts[wid] = __popc(bal);
            __syncthreads();
            int off = total;
            for (int w = 0; w < wid; ++w) off += warp_counts[w];
            if (c) {
                const int r = off + __popc(bal & ((1u << ln) - 1u));
                rows[r] = slot * rows_per_seq + (i - pos0);
                rows_out[r] = b * L + i;
            }
            __syncthreads();
            if (tid == 0) {
                int t = 0;
                for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += warp_counts[w];
                total += t;
            }
            __syncthreads();
        }
    }
    if (tid == 0) *d_R = total;
}

// Merge the per-chunk partial statistics of each active row and scatter them to the [B, L] outputs.
// The merge is associative and symmetric (equal maxima resolve to the lower token id), so one warp per
// row lets its lanes take chunks round-robin and then combines them with a butterfly.
struct StatTuple {
    float m1, m2, S;
    int i1;
};
__device__ __forceinline__ StatTuple merge_tuples(const StatTuple& a, const StatTuple& b) {
    StatTuple r;
    r.m1 = fmaxf(a.m1, b.m1);
    r.m2 = fmaxf(fmaxf(a.m2, b.m2), fminf(a.m1, b.m1));
    const float sa = (a.m1 == -INFINITY) ? 0.f : a.S * expf(a.m1 - r.m1);
    const float sb = (b.m1 == -INFINITY) ? 0.f : b.S * expf(b.m1 - r.m1);
    r.S = sa + sb;
    r.i1 = (b.m1 > a.m1 || (b.m1 == a.m1 && b.i1 < a.i1)) ? b.i1 : a.i1;
    return r;
}
__global__ void __launch_bounds__(128) merge_stats_kernel(const float4* __restrict__ partials, int R_pad, int grid_gemm,
                                                          int n_vt, int pair_mode, const int32_t* __restrict__ rows,
                                                          const int32_t* __restrict__ d_R, float* __restrict__ top1,
                                                          float* __restrict__ top2, float* __restrict__ sumexp,
                                                          int32_t* __restrict__ argmax,
                                                          const float2* __restrict__ partials2,
                                                          int32_t* __restrict__ sampled) {
    grid_launch_dependents();
    grid_dependency_wait();
    const int R = *d_R;
    const int r = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (r >= R) return;
    // the same split of the vocabulary into chunks as the kernel that wrote the partial tuples
    const int n_rb = (R + 127) / 128;
    int n_ch = pair_mode ? (grid_gemm / 2) / ((n_rb + 1) / 2) : grid_gemm / n_rb;
    if (n_ch > n_vt) n_ch = n_vt;
    StatTuple t{-INFINITY, -INFINITY, 0.f, 0x7fffffff};
    for (int c = lane; c < n_ch; c += 32) {
        const float4 v = partials[(size_t)c * R_pad + r];
        t = merge_tuples(t, StatTuple{v.x, v.z, v.w, __float_as_int(v.y)});
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        StatTuple u;
        u.m1 = __shfl_xor_sync(0xffffffffu, t.m1, o);
        u.m2 = __shfl_xor_sync(0xffffffffu, t.m2, o);
        u.S = __shfl_xor_sync(0xffffffffu, t.S, o);
        u.i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
        t = merge_tuples(t, u);
    }
    if (partials2) {
        // the Gumbel-max draw: largest perturbed score over the chunks, the lower token id on a tie
        float best = -INFINITY;
        int best_i = 0x7fffffff;
        for (int c = lane; c < n_ch; c += 32) {
            const float2 v = partials2[(size_t)c * R_pad + r];
            const int vi = __float_as_int(v.y);
            if (v.x > best || (v.x == best && vi < best_i)) { best = v.x; best_i = vi; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
            if (ob > best || (ob == best && oi < best_i)) { best = ob; best_i = oi; }
        }
        if (lane == 0) sampled[rows[r]] = best_i;
    }
    if (lane == 0) {
        const int flat = rows[r];
        top1[flat] = t.m1;
        top2[flat] = t.m2;
        sumexp[flat] = t.S;
        argmax[flat] = t.i1;
    }
}

// Statistics of the same rows over two disjoint parts of the vocabulary -> statistics over their union, element by
// element over [n] arrays (the rule merge_stats_kernel applies to the chunks of one launch): what a rank does with
// the tuples its peers computed on their vocabulary slices.  out may alias a.
__global__ void merge_stat_arrays_kernel(int n, const float* __restrict__ a1, const float* __restrict__ a2,
                                         const float* __restrict__ aS, const int32_t* __restrict__ ai,
                                         const float* __restrict__ b1, const float* __restrict__ b2,
                                         const float* __restrict__ bS, const int32_t* __restrict__ bi, float* o1,
                                         float* o2, float* oS, int32_t* oi) {
    grid_launch_dependents();
    grid_dependency_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const StatTuple t = merge_tuples(StatTuple{a1[i], a2[i], aS[i], ai[i]}, StatTuple{b1[i], b2[i], bS[i], bi[i]});
    o1[i] = t.m1;
    o2[i] = t.m2;
    oS[i] = t.S;
    oi[i] = t.i1;
}

// Sequences that still have work, in ascending order: seq_map[slot] = b, the remaining slots -1,
// *n_active = count.  One warp.
__global__ void build_seq_map_kernel(const SeqState* __restrict__ state, int B, int n_blocks,
                                     int32_t* __restrict__ seq_map, int32_t* __restrict__ n_active) {
    grid_launch_dependents();
    grid_dependency_wait();
    const int ln = threadIdx.x;
    int total = 0;
    for (int base = 0; base < B; base += 32) {
        const int b = base + ln;
        const bool live = b < B && state[b].blk < n_blocks;
        const uint32_t bal = __ballot_sync(0xffffffffu, live);
        if (live) seq_map[total + __popc(bal & ((1u << ln) - 1u))] = b;
        total += __popc(bal);
    }
    for (int slot = total + ln; slot < B; slot += 32) seq_map[slot] = -1;
    if (ln == 0) *n_active = total;
}

// x = [prompt ; mask_id * G]  and fresh loop state  (Algorithm 1, initialisation)
__global__ void init_canvas_kernel(const int32_t* __restrict__ prompt, int32_t* __restrict__ x, int B, int P, int G,
                                   int32_t mask_id, SeqState* __restrict__ state) {
    grid_launch_dependents();
    grid_dependency_wait();
    const int L = P + G;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < B * L) {
        const int b = idx / L, i = idx % L;
        x[idx] = (i < P) ? prompt[(size_t)b * P + i] : mask_id;
    }
    if (idx < B) state[idx] = SeqState{0, 0, 0, G > 0 ? 1 : 0};
}

}  // namespace jot
