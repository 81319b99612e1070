// C ABI of the JoT denoising-step library: argument checks, workspace layout, tensor maps, kernel
// launches and the generate loop of Algorithm 1.  All arithmetic of the step lives in the kernels
// (gemm.cuh, attention.cuh, glue.cuh, accept.cuh); nothing here computes on the host.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstddef>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/jot.h"
#include "accept.cuh"
#include "attention.cuh"
#include "gemm.cuh"
#include "gemm2.cuh"
#include "gemm_slab.cuh"
#include "glue.cuh"

using namespace jot;

namespace {

thread_local int g_last_cuda_error = 0;
std::atomic<int64_t> g_launches{0};

#define JOT_CUDA(expr)                                  \
    do {                                                \
        cudaError_t e_ = (expr);                        \
        if (e_ != cudaSuccess) {                        \
            g_last_cuda_error = (int)e_;                \
            return JOT_ERR_CUDA;                        \
        }                                               \
    } while (0)
#define JOT_TRY(expr)              \
    do {                           \
        int s_ = (expr);           \
        if (s_ != JOT_OK) return s_; \
    } while (0)

inline int launch_check() {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return JOT_ERR_CUDA;
    }
    return JOT_OK;
}

// Every kernel goes out through here: programmatic stream serialization lets a kernel's launch and
// on-chip prologue overlap the tail of its predecessor (see pdl.cuh for the device side).
template <typename... KArgs, typename... Args>
void launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);     // errors are picked up by launch_check()
}

// ---------------------------------------------------------------- device facts
struct DeviceInfo {
    int ok = 0, sms = 0, status = JOT_OK;
    PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
};

int device_info(DeviceInfo** out) {
    static thread_local DeviceInfo cache[64];
    int dev = 0;
    JOT_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return JOT_ERR_DEVICE;
    DeviceInfo& di = cache[dev];
    if (!di.ok) {
        int major = 0;
        JOT_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        JOT_CUDA(cudaDeviceGetAttribute(&di.sms, cudaDevAttrMultiProcessorCount, dev));
        if (major != 10) return JOT_ERR_DEVICE;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        JOT_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return JOT_ERR_DEVICE;
        di.encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
        di.ok = 1;
    }
    *out = &di;
    return JOT_OK;
}

// bf16 row-major [rows, cols] (row stride ld elements), boxes of 64 columns x box_rows rows, 128-byte swizzle;
// out-of-range elements read as zero.
int make_map_2d(const DeviceInfo* di, CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld,
                uint32_t box_rows) {
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = di->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error = (int)cudaErrorInvalidValue;
        return JOT_ERR_CUDA;
    }
    return JOT_OK;
}
// qkv viewed as (column, position, sequence)
int make_map_qkv(const DeviceInfo* di, CUtensorMap* map, const void* ptr, uint64_t B, uint64_t L, uint64_t cols) {
    cuuint64_t dims[3] = {cols, L, B};
    cuuint64_t strides[2] = {cols * 2, L * cols * 2};
    cuuint32_t box[3] = {64, 128, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = di->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_last_cuda_error = (int)cudaErrorInvalidValue;
        return JOT_ERR_CUDA;
    }
    return JOT_OK;
}

// ---------------------------------------------------------------- GEMM launch
template <int BN, int EPI>
int launch_gemm_t(const GemmParams& p, const CUtensorMap& tmA, const CUtensorMap& tmB, int grid, cudaStream_t st) {
    static thread_local bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev & 63]) {
        JOT_CUDA(cudaFuncSetAttribute(gemm_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      GemmSmem<BN>::DYN_BYTES));
        attr_set[dev & 63] = true;
    }
    launch_k((gemm_kernel<BN, EPI>), dim3(grid), dim3(kGemmThreads), GemmSmem<BN>::DYN_BYTES, st, p, tmA, tmB);
    return launch_check();
}

template <int EPI>
int launch_pair_t(const GemmParams& p, const CUtensorMap& tmA, const CUtensorMap& tmB, int grid, cudaStream_t st) {
    static thread_local bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev & 63]) {
        JOT_CUDA(cudaFuncSetAttribute(gemm_pair_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairDynBytes));
        attr_set[dev & 63] = true;
    }
    launch_k((gemm_pair_kernel<EPI>), dim3(grid & ~1), dim3(kGemmThreads), kPairDynBytes, st, p, tmA, tmB);
    return launch_check();
}

struct WeightMaps {     // one weight matrix as B operand, for both tile widths
    CUtensorMap m128, m256;
};

int make_weight_maps(const DeviceInfo* di, WeightMaps* w, const void* ptr, int rows, int cols, bool swiglu) {
    // swiglu tiles fetch gate and up rows as two boxes of half the tile width
    JOT_TRY(make_map_2d(di, &w->m128, ptr, rows, cols, cols, swiglu ? 64 : 128));
    JOT_TRY(make_map_2d(di, &w->m256, ptr, rows, cols, cols, swiglu ? 128 : 256));
    return JOT_OK;
}

// ---------------------------------------------------------------- slab kernel (canvases of at most 512 rows)
// A token matrix [M, K] as the slab kernel's N operand: one box shape per accumulator (half its tokens).
struct SlabMaps {
    CUtensorMap x0, x1;
};
int make_slab_maps(const DeviceInfo* di, SlabMaps* sm, const void* ptr, int M, int K, int ld) {
    const SlabGeom g = slab_geom(M, 1);
    JOT_TRY(make_map_2d(di, &sm->x0, ptr, M, K, ld, (uint32_t)(g.n0 / 2)));
    JOT_TRY(make_map_2d(di, &sm->x1, ptr, M, K, ld, (uint32_t)(g.n1 ? g.n1 / 2 : g.n0 / 2)));
    return JOT_OK;
}

// Clusters of `split` CTA pairs; the launch covers pair-slabs slab0 .. slab0 + n_slabs - 1.
template <int EPI>
int launch_slab_t(GemmParams p, const CUtensorMap& tmW, const SlabMaps& tmX, int slab0, int n_slabs, int split,
                  cudaStream_t st) {
    static thread_local bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev & 63]) {
        JOT_CUDA(cudaFuncSetAttribute(gemm_slab_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSlabMaxSmem));
        attr_set[dev & 63] = true;
    }
    p.slab0 = slab0;
    p.slab_split = split;
    const SlabGeom g = slab_geom(p.M, split);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(n_slabs * 2 * split));
    cfg.blockDim = dim3(kSlabThreads);
    cfg.dynamicSmemBytes = (size_t)g.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)(2 * split);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaLaunchKernelEx(&cfg, gemm_slab_kernel<EPI>, p, tmW, tmX.x0, tmX.x1);
    return launch_check();
}

// Gate/up + SwiGLU for canvases of 353 .. 384 rows: one launch, two units of work per pair (gemm_slab.cuh).
int launch_slab_gateup2(GemmParams p, const CUtensorMap& tmW, const SlabMaps& tmX, const Slab2Plan& plan, cudaStream_t st) {
    static thread_local bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev & 63]) {
        JOT_CUDA(cudaFuncSetAttribute(gemm_slab_gateup2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSlab2Smem));
        attr_set[dev & 63] = true;
    }
    p.slab0 = plan.A;
    p.slab_split = plan.G;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * plan.A));
    cfg.blockDim = dim3(kSlabThreads);
    cfg.dynamicSmemBytes = (size_t)kSlab2Smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaLaunchKernelEx(&cfg, gemm_slab_gateup2_kernel, p, tmW, tmX.x0, tmX.x1);
    return launch_check();
}

// How many clusters of `split` pairs the device runs side by side (1 CTA per SM: the kernel takes all shared memory).
int slab_cluster_capacity(int sms, int split) {
    static thread_local int cap[64][5] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    int& c = cap[dev & 63][split];
    if (c == 0) {
        cudaFuncSetAttribute(gemm_slab_kernel<SLAB_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSlabMaxSmem);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(2 * split * 64));
        cfg.blockDim = dim3(kSlabThreads);
        cfg.dynamicSmemBytes = (size_t)kSlabMaxSmem - 1024;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)(2 * split);
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_slab_kernel<SLAB_STORE>, &cfg) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            n = sms / (2 * split) * 3 / 4;          // a guess that errs on the low side
        }
        c = n > 0 ? n : 1;
    }
    return c;
}

// Largest K split (pairs per cluster) that keeps `n_slabs` clusters in one wave, leaves every pair at least 8
// k-blocks and fits the reduce-scatter buffers in shared memory.
int slab_pick_split(int M, int n_slabs, int num_kb, int sms) {
    for (int s = 4; s > 1; --s) {
        if (num_kb / s < 8) continue;
        if (slab_geom(M, s).smem_bytes > kSlabMaxSmem) continue;
        if (n_slabs <= slab_cluster_capacity(sms, s)) return s;
    }
    return 1;
}

int run_slab(const DeviceInfo* di, const SlabMaps& tmX, const WeightMaps& w, int epi, const GemmParams& p, cudaStream_t st) {
    const int n_out = (epi == EPI_SWIGLU) ? p.N / 2 : p.N;
    const int per_slab = (epi == EPI_SWIGLU) ? 128 : 256;                 // output features per CTA pair
    const int n_slabs = (n_out + per_slab - 1) / per_slab;
    const int num_kb = (p.K + kBK - 1) / kBK;
    auto go = [&](int slab0, int n, int split) -> int {
        if (n <= 0) return JOT_OK;
        if (epi == EPI_STORE) return launch_slab_t<SLAB_STORE>(p, w.m128, tmX, slab0, n, split, st);
        if (epi == EPI_QKV) return launch_slab_t<SLAB_QKV>(p, w.m128, tmX, slab0, n, split, st);
        return launch_slab_t<SLAB_SWIGLU>(p, w.m128, tmX, slab0, n, split, st);
    };
    const int cap1 = slab_cluster_capacity(di->sms, 1);
    if (epi == EPI_SWIGLU && p.N % 256 == 0) {
        const Slab2Plan plan = slab2_plan(p.M, n_slabs, cap1);
        if (plan.ok) return launch_slab_gateup2(p, w.m128, tmX, plan, st);
    }
    // whole waves of unsplit slabs first; what is left over (or a projection with few slabs) is cut along K so
    // that it still fills the machine
    const int full = n_slabs / cap1 * cap1, rest = n_slabs - full;
    JOT_TRY(go(0, full, 1));
    return go(full, rest, slab_pick_split(p.M, rest, num_kb, di->sms));
}

// Which kernel shape moves the fewest operand bytes through an SM for this projection: waves x bytes per
// k-block (48 KB for a 128 x 256 tile, 32 KB for a 128 x 128 tile, 32 KB per CTA of a 256 x 256 pair tile).
enum { SHAPE_256 = 0, SHAPE_128 = 1, SHAPE_PAIR = 2 };
int pick_shape(int M, int n_out, int sms, bool allow_128) {
    const long m_blks = (M + 127) / 128, n256 = (n_out + 255) / 256, n128 = (n_out + 127) / 128;
    auto waves = [](long tiles, long slots) { return (tiles + slots - 1) / slots; };
    const long c256 = waves(m_blks * n256, sms) * 48;
    const long c128 = allow_128 ? waves(m_blks * n128, sms) * 32 : (1L << 60);
    const long cpair = m_blks >= 2 ? waves(((m_blks + 1) / 2) * n256, sms / 2) * 32 : (1L << 60);
    if (c256 <= c128 && c256 <= cpair) return SHAPE_256;
    return cpair <= c128 ? SHAPE_PAIR : SHAPE_128;
}

// Split-K factor for a plain projection: when 256-wide tiles leave most SMs idle, cut K into up to 4
// ranges so that (tiles x ranges) still fits one wave.  Needs `scratch` for the fp32 partial sums.
int pick_split(int M, int N, int K, int sms, size_t scratch_bytes) {
    const long tiles = (long)((M + 127) / 128) * ((N + 255) / 256);
    const int num_kb = (K + kBK - 1) / kBK;
    int split = (int)(sms / tiles);
    if (split > 4) split = 4;
    while (split > 1 && (num_kb / split < 8 || (size_t)split * M * N * 4 > scratch_bytes)) --split;
    return split < 1 ? 1 : split;
}

// An RMSNorm that directly follows a projection; when the projection goes through split-K the norm is
// folded into the kernel that adds the K ranges (`done` reports whether that happened).
struct NormAfter {
    const __nv_bfloat16* gain;
    __nv_bfloat16* out;
    float eps;
    bool done;
};

int run_gemm(const DeviceInfo* di, const CUtensorMap& tmA, const WeightMaps& w, int epi, GemmParams p, cudaStream_t st,
             float* scratch = nullptr, size_t scratch_bytes = 0, NormAfter* norm = nullptr,
             const SlabMaps* tmX_slab = nullptr) {
    // small canvases: weight rows as the MMA's M side, every token in tensor memory (gemm_slab.cuh)
    if (tmX_slab && p.M <= kSlabMaxTokens) return run_slab(di, *tmX_slab, w, epi, p, st);      // callers decide when
    if (epi == EPI_STORE && scratch) {
        const int split = pick_split(p.M, p.N, p.K, di->sms, scratch_bytes);
        if (split > 1) {
            p.split_k = split;
            p.partial = scratch;
            const long items = (long)((p.M + 127) / 128) * ((p.N + 255) / 256) * split;
            JOT_TRY((launch_gemm_t<256, EPI_PARTIAL>(p, tmA, w.m256, (int)items, st)));
            if (norm && p.ldc == p.N && p.N / 8 <= 1024) {
                int threads = (p.N / 8 + 31) / 32 * 32;      // one 8-element vector per thread up to 512 threads
                threads = threads > 512 ? 512 : (threads < 64 ? 64 : threads);
                launch_k(splitk_reduce_norm_kernel, dim3(p.M), dim3(threads), 0, st, scratch, split, p.residual, p.C, p.M,
                         p.N, norm->gain, norm->out, norm->eps);
                norm->done = true;
                return launch_check();
            }
            const size_t n8 = (size_t)p.M * p.N / 8;
            launch_k(splitk_reduce_kernel, dim3((unsigned)((n8 + 255) / 256)), dim3(256), 0, st, scratch, split, p.residual, p.C, p.M, p.N);
            return launch_check();
        }
    }
    // for SwiGLU a "256-wide" tile holds 128 gate + 128 up columns, i.e. 128 output columns
    const int n_out = (epi == EPI_SWIGLU) ? p.N / 2 : p.N;
    const int n_eff = (epi == EPI_SWIGLU) ? 2 * n_out : n_out;
    const int shape = pick_shape(p.M, n_eff, di->sms, true);
    if (shape == SHAPE_PAIR) {
        const long tiles = (long)(((p.M + 127) / 128 + 1) / 2) * ((n_eff + 255) / 256);
        const int grid = (int)(2 * tiles < di->sms ? 2 * tiles : di->sms);
        // each CTA of a pair fetches 128 rows of W: the 128-row box of the plain maps, the 128-row box of SwiGLU's
        if (epi == EPI_STORE) return launch_pair_t<EPI_STORE>(p, tmA, w.m128, grid, st);
        if (epi == EPI_QKV) return launch_pair_t<EPI_QKV>(p, tmA, w.m128, grid, st);
        return launch_pair_t<EPI_SWIGLU>(p, tmA, w.m256, grid, st);
    }
    const int bn = shape == SHAPE_128 ? 128 : 256;
    const int bn_out = (epi == EPI_SWIGLU) ? bn / 2 : bn;
    long tiles = (long)((p.M + 127) / 128) * ((n_out + bn_out - 1) / bn_out);
    int grid = (int)(tiles < di->sms ? tiles : di->sms);
    if (grid <= 0) return JOT_OK;
    if (epi == EPI_STORE)
        return bn == 256 ? launch_gemm_t<256, EPI_STORE>(p, tmA, w.m256, grid, st)
                         : launch_gemm_t<128, EPI_STORE>(p, tmA, w.m128, grid, st);
    if (epi == EPI_QKV)
        return bn == 256 ? launch_gemm_t<256, EPI_QKV>(p, tmA, w.m256, grid, st)
                         : launch_gemm_t<128, EPI_QKV>(p, tmA, w.m128, grid, st);
    return bn == 256 ? launch_gemm_t<256, EPI_SWIGLU>(p, tmA, w.m256, grid, st)
                     : launch_gemm_t<128, EPI_SWIGLU>(p, tmA, w.m128, grid, st);
}

template <int HD>
int launch_attention_t(const AttnParams& p, const CUtensorMap& tq, const CUtensorMap& tv, dim3 grid, cudaStream_t st) {
    static thread_local bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set[dev & 63]) {
        JOT_CUDA(cudaFuncSetAttribute(attention_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      AttnSmem<HD>::DYN_BYTES));
        attr_set[dev & 63] = true;
    }
    launch_k((attention_kernel<HD>), dim3(grid), dim3(kAttnThreads), AttnSmem<HD>::DYN_BYTES, st, p, tq, tv);
    return launch_check();
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

// ---------------------------------------------------------------- model object
struct jot_model {
    jot_model_config cfg;
    int max_batch, max_seq;
    DeviceInfo di_val;    // a copy: the model may outlive the thread that created it
    DeviceInfo* di;
    bool sync_steps = true;    // single-step entry points read the status word before they return
    // borrowed weights
    const __nv_bfloat16 *embed, *lm_head, *final_norm;
    std::vector<const __nv_bfloat16*> attn_norm, mlp_norm;
    std::vector<WeightMaps> wqkv, wo, wgu, wdown;
    WeightMaps wlm;
    // workspace slices
    int32_t* ctrl;        // [0] status, [1] R, [2] n_unfinished
    float2* rope_cs;
    __nv_bfloat16 *h, *a, *qkv, *vt, *attn, *act, *hsel;
    int32_t *rows, *rows_out, *seq_map;
    float4* partials;
    float2* partials2;
    int32_t* g_sampled;
    float* splitk;
    int R_cap;
    int32_t* canvas;      // generate: tokens [max_batch * max_seq]
    float *g_top1, *g_top2, *g_sumexp;
    int32_t* g_argmax;
    SeqState* state;
    AcceptParamsDev* params_dev;
    // activation tensor maps, re-encoded when (B, L) changes
    int map_B = -1, map_L = -1;
    CUtensorMap tm_hsel, tm_qkv3, tm_vt;
    // A-operand maps of the projections for a pass over M rows (rows past M read as zero without memory
    // traffic): one set for the whole canvas, one for the rows of a block
    // (x*: the same buffers as the token operand of the slab kernel, boxes of half an accumulator's tokens)
    struct ActMaps { int M = -1; bool slab = false, slab_gate_up = false; CUtensorMap a, attn, act; SlabMaps xa, xattn, xact; };
    ActMaps maps_full, maps_span;
    // block-wise KV cache (caller's memory, optional): per layer the rotated Q/K rows and V^T of the whole canvas
    uint8_t* kv_base = nullptr;
    size_t kv_bytes = 0;
    std::vector<__nv_bfloat16*> kv_qkv, kv_vt;
    std::vector<CUtensorMap> kv_tm_qkv3, kv_tm_vt;
    int kv_map_B = -1, kv_map_L = -1;       // geometry the per-layer maps were encoded for
    int kv_valid_B = -1, kv_valid_L = -1;   // geometry of the last refresh (block passes need one)
    int32_t* h_pinned = nullptr;    // pinned host words for loop control read-back (two 4-word slots, then SeqState)
    cudaEvent_t step_done[2] = {nullptr, nullptr};
    // optional per-kernel-class timing with CUDA events on the launching stream
    bool profiling = false;
    std::vector<cudaEvent_t> ev_pool;
    size_t ev_used = 0;
    struct Span { int cls; cudaEvent_t a, b; };
    std::vector<Span> spans;
    double prof_ms[JOT_PROF_CLASSES] = {};
    int64_t prof_n[JOT_PROF_CLASSES] = {};
};

namespace {

// Brackets one kernel launch with a pair of events while profiling is on.
struct ProfScope {
    jot_model* m;
    cudaStream_t st;
    cudaEvent_t b = nullptr;
    int cls;
    ProfScope(jot_model* m_, int cls_, cudaStream_t st_) : m(m_), st(st_), cls(cls_) {
        if (!m->profiling) return;
        cudaEvent_t a = next();
        b = next();
        if (a && b) {
            cudaEventRecord(a, st);
            m->spans.push_back({cls, a, b});
        }
    }
    ~ProfScope() {
        if (b) cudaEventRecord(b, st);
    }
    cudaEvent_t next() {
        if (m->ev_used == m->ev_pool.size()) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
            m->ev_pool.push_back(e);
        }
        return m->ev_pool[m->ev_used++];
    }
};

struct Layout {
    size_t ctrl, rope, h, a, qkv, vt, attn, act, hsel, rows, rows_out, seq_map, partials, partials2, sampled, splitk, canvas, top1, top2, sumexp, argmax, state, params,
        total;
};

constexpr size_t kSplitKBytes = (size_t)148 * 128 * 256 * 4 + 4096;   // one wave of 128 x 256 fp32 tiles

bool config_ok(const jot_model_config* c) {
    if (!c) return false;
    if (c->n_layers < 0 || c->d_model <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->d_ff <= 0 || c->vocab <= 1)
        return false;
    if (c->head_dim != 64 && c->head_dim != 128) return false;
    if (c->d_model % 64 || c->d_ff % 64 || c->vocab % 8 || c->n_q_heads % c->n_kv_heads) return false;
    if (c->d_model > 16384) return false;
    if (c->mask_id < 0 || c->mask_id >= c->vocab) return false;
    return true;
}

Layout make_layout(const jot_model_config* c, int max_batch, int max_seq) {
    Layout l;
    const size_t M = (size_t)max_batch * max_seq, R_cap = align_up(M, 128);
    const size_t qkv_cols = (size_t)(c->n_q_heads + 2 * c->n_kv_heads) * c->head_dim;
    const size_t Lp = align_up((size_t)max_seq, 8);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off = align_up(off + bytes, 1024);
        return o;
    };
    l.ctrl = take(1024);
    l.rope = take((size_t)max_seq * (c->head_dim / 2) * sizeof(float2));
    l.h = take(M * c->d_model * 2);
    l.a = take(M * c->d_model * 2);
    l.qkv = take(M * qkv_cols * 2);
    l.vt = take((size_t)max_batch * c->n_kv_heads * c->head_dim * Lp * 2);
    l.attn = take(M * (size_t)c->n_q_heads * c->head_dim * 2);
    l.act = take(M * (size_t)c->d_ff * 2);
    l.hsel = take(R_cap * c->d_model * 2);
    l.rows = take(R_cap * 4);
    l.rows_out = take(R_cap * 4);
    l.seq_map = take((size_t)max_batch * 4);
    l.partials = take((size_t)256 * R_cap * sizeof(float4));   // up to 256 vocabulary chunks
    l.partials2 = take((size_t)256 * R_cap * sizeof(float2));
    l.sampled = take(M * 4);
    l.splitk = take(kSplitKBytes);
    l.canvas = take(M * 4);
    l.top1 = take(M * 4);
    l.top2 = take(M * 4);
    l.sumexp = take(M * 4);
    l.argmax = take(M * 4);
    l.state = take((size_t)max_batch * sizeof(SeqState));
    l.params = take((size_t)max_batch * sizeof(AcceptParamsDev));
    l.total = off;
    return l;
}

int encode_activation_maps(jot_model* m, int B, int L) {
    if (m->map_B == B && m->map_L == L) return JOT_OK;
    const jot_model_config& c = m->cfg;
    const int M = B * L;
    const int qkv_cols = (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
    const int Lp = (int)align_up((size_t)L, 8);
    (void)M;
    JOT_TRY(make_map_2d(m->di, &m->tm_hsel, m->hsel, m->R_cap, c.d_model, c.d_model, 128));
    JOT_TRY(make_map_qkv(m->di, &m->tm_qkv3, m->qkv, B, L, qkv_cols));
    JOT_TRY(make_map_2d(m->di, &m->tm_vt, m->vt, (uint64_t)B * c.n_kv_heads * c.head_dim, L, Lp, c.head_dim));
    m->map_B = B;
    m->map_L = L;
    return JOT_OK;
}

int encode_act_maps(jot_model* m, jot_model::ActMaps* am, int M) {
    if (am->M == M) return JOT_OK;
    const jot_model_config& c = m->cfg;
    JOT_TRY(make_map_2d(m->di, &am->a, m->a, M, c.d_model, c.d_model, 128));
    JOT_TRY(make_map_2d(m->di, &am->attn, m->attn, M, c.n_q_heads * c.head_dim, c.n_q_heads * c.head_dim, 128));
    JOT_TRY(make_map_2d(m->di, &am->act, m->act, M, c.d_ff, c.d_ff, 128));
    am->slab = M <= kSlabPreferTokens;
    am->slab_gate_up = (M > 128 && M <= kSlabGateUpTokens) ||
                       ((2 * c.d_ff) % 256 == 0 &&
                        slab2_plan(M, 2 * c.d_ff / 256, slab_cluster_capacity(m->di->sms, 1)).ok);
    if (am->slab || am->slab_gate_up) {
        JOT_TRY(make_slab_maps(m->di, &am->xa, m->a, M, c.d_model, c.d_model));
        JOT_TRY(make_slab_maps(m->di, &am->xattn, m->attn, M, c.n_q_heads * c.head_dim, c.n_q_heads * c.head_dim));
        JOT_TRY(make_slab_maps(m->di, &am->xact, m->act, M, c.d_ff, c.d_ff));
    }
    am->M = M;
    return JOT_OK;
}

// Per-layer slices of an attached KV cache for canvases of B x L, and their tensor maps.
size_t kv_layer_bytes(const jot_model_config* c, int max_batch, int max_seq, size_t* vt_off) {
    const size_t qkv_cols = (size_t)(c->n_q_heads + 2 * c->n_kv_heads) * c->head_dim;
    const size_t q = align_up((size_t)max_batch * max_seq * qkv_cols * 2, 1024);
    const size_t v = align_up((size_t)max_batch * c->n_kv_heads * c->head_dim * align_up((size_t)max_seq, 8) * 2, 1024);
    if (vt_off) *vt_off = q;
    return q + v;
}

int encode_kv_maps(jot_model* m, int B, int L) {
    if (m->kv_map_B == B && m->kv_map_L == L) return JOT_OK;
    const jot_model_config& c = m->cfg;
    const int qkv_cols = (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
    const int Lp = (int)align_up((size_t)L, 8);
    for (int l = 0; l < c.n_layers; ++l) {
        JOT_TRY(make_map_qkv(m->di, &m->kv_tm_qkv3[l], m->kv_qkv[l], B, L, qkv_cols));
        JOT_TRY(make_map_2d(m->di, &m->kv_tm_vt[l], m->kv_vt[l], (uint64_t)B * c.n_kv_heads * c.head_dim, L, Lp, c.head_dim));
    }
    m->kv_map_B = B;
    m->kv_map_L = L;
    m->kv_valid_B = m->kv_valid_L = -1;      // another geometry lays the rows out differently
    return JOT_OK;
}

// Which rows a pass covers: positions pos0 .. pos0 + Lr - 1 of every sequence; use_cache: the rotated Q/K
// rows and V^T of every layer live in the attached KV cache instead of the one scratch buffer, so that a
// later pass over one block finds the rest of the canvas there.
struct FwdSpan {
    int Lr, pos0;
    bool use_cache;
};

// Transformer body: tokens [B, L] -> residual stream m->h [B*Lr, d] (before the final norm).
// B sequences are processed; with seq_map they are the compacted batch (slot -> sequence of d_tokens).
int forward_body(jot_model* m, const int32_t* d_tokens, int B, int L, cudaStream_t st, const int32_t* seq_map = nullptr,
                 const FwdSpan* span = nullptr) {
    const jot_model_config& c = m->cfg;
    const int Lr = span ? span->Lr : L, pos0 = span ? span->pos0 : 0;
    const bool cached = span && span->use_cache;
    const int M = B * Lr, d = c.d_model, hd = c.head_dim, nq = c.n_q_heads, nkv = c.n_kv_heads;
    const int qkv_cols = (nq + 2 * nkv) * hd;
    const int Lp = (int)align_up((size_t)L, 8);
    JOT_TRY(encode_activation_maps(m, B, L));
    jot_model::ActMaps& am = (Lr == L) ? m->maps_full : m->maps_span;
    JOT_TRY(encode_act_maps(m, &am, M));
    if (cached) JOT_TRY(encode_kv_maps(m, B, L));
    int32_t* status = m->ctrl;

    {
        ProfScope ps(m, JOT_PROF_EMBED, st);
        launch_k(embed_kernel, dim3(M), dim3(128), 0, st, d_tokens, m->embed, m->h, d, L, seq_map, Lr, pos0, c.vocab, status);
    }
    JOT_TRY(launch_check());
    bool norm_ready = false;          // true when a fused split-K tail has already written the next norm into m->a
    for (int l = 0; l < c.n_layers; ++l) {
        if (!norm_ready) {
            ProfScope ps(m, JOT_PROF_RMSNORM, st);
            launch_k(rmsnorm_kernel, dim3(M), dim3(256), 0, st, m->h, m->attn_norm[l], m->a, d, c.rms_eps, nullptr, nullptr);
            JOT_TRY(launch_check());
        }
        GemmParams p{};
        p.M = M; p.N = qkv_cols; p.K = d; p.C = cached ? m->kv_qkv[l] : m->qkv; p.ldc = qkv_cols; p.status = status;
        {
            ProfScope ps(m, JOT_PROF_GEMM_QKV, st);
            p.vt = cached ? m->kv_vt[l] : m->vt; p.rope_cs = m->rope_cs; p.L = L; p.Lp = Lp; p.nq = nq; p.nkv = nkv;
            p.hd = hd; p.rows_per_seq = Lr; p.pos0 = pos0;
            JOT_TRY(run_gemm(m->di, am.a, m->wqkv[l], EPI_QKV, p, st, nullptr, 0, nullptr, am.slab ? &am.xa : nullptr));
        }
        AttnParams ap{};
        ap.B = B; ap.L = L; ap.nq = nq; ap.nkv = nkv; ap.out = m->attn; ap.status = status;
        ap.q_lo = pos0; ap.q_cnt = Lr;
        ap.scale_log2e = 1.4426950408889634f / sqrtf((float)hd);
        const long items = (long)B * nq * ((Lr + 127) / 128);
        dim3 grid((unsigned)(items < m->di->sms ? items : m->di->sms));
        {
            ProfScope ps(m, JOT_PROF_ATTENTION, st);
            const CUtensorMap& tq = cached ? m->kv_tm_qkv3[l] : m->tm_qkv3;
            const CUtensorMap& tv = cached ? m->kv_tm_vt[l] : m->tm_vt;
            if (hd == 128) JOT_TRY(launch_attention_t<128>(ap, tq, tv, grid, st));
            else JOT_TRY(launch_attention_t<64>(ap, tq, tv, grid, st));
        }
        p = GemmParams{};
        p.M = M; p.N = d; p.K = nq * hd; p.C = m->h; p.residual = m->h; p.ldc = d; p.status = status;
        {
            ProfScope ps(m, JOT_PROF_GEMM_O, st);
            NormAfter na{m->mlp_norm[l], m->a, c.rms_eps, false};
            JOT_TRY(run_gemm(m->di, am.attn, m->wo[l], EPI_STORE, p, st, m->splitk, kSplitKBytes, &na,
                             am.slab ? &am.xattn : nullptr));
            norm_ready = na.done;
        }
        if (!norm_ready) {
            ProfScope ps(m, JOT_PROF_RMSNORM, st);
            launch_k(rmsnorm_kernel, dim3(M), dim3(256), 0, st, m->h, m->mlp_norm[l], m->a, d, c.rms_eps, nullptr, nullptr);
            JOT_TRY(launch_check());
        }
        p = GemmParams{};
        p.M = M; p.N = 2 * c.d_ff; p.K = d; p.C = m->act; p.ldc = c.d_ff; p.status = status;
        {
            ProfScope ps(m, JOT_PROF_GEMM_GATE_UP, st);
            // (up to 128 rows the token-major tiles stream the gate/up weights faster than the slab kernel's two
            // launches do: measured 39-43 us against 42-47)
            JOT_TRY(run_gemm(m->di, am.a, m->wgu[l], EPI_SWIGLU, p, st, nullptr, 0, nullptr,
                             am.slab_gate_up ? &am.xa : nullptr));
        }
        p = GemmParams{};
        p.M = M; p.N = d; p.K = c.d_ff; p.C = m->h; p.residual = m->h; p.ldc = d; p.status = status;
        {
            ProfScope ps(m, JOT_PROF_GEMM_DOWN, st);
            NormAfter na{l + 1 < c.n_layers ? m->attn_norm[l + 1] : nullptr, m->a, c.rms_eps, false};
            JOT_TRY(run_gemm(m->di, am.act, m->wdown[l], EPI_STORE, p, st, m->splitk, kSplitKBytes,
                             na.gain ? &na : nullptr, am.slab ? &am.xact : nullptr));
            norm_ready = na.done;
        }
    }
    return JOT_OK;
}

// hsel (active rows, already gathered) -> merged statistics scattered to the [B, L] outputs
// Sampling-based finalisation of the head: temperature > 0 turns it on; the step index of a row is its
// sequence's own count of denoising steps so far when d_seq_steps is given (generate loop: the draw then does
// not depend on what else is in the batch), else step_value.
struct HeadSampling {
    float temperature = 0.f;
    unsigned long long seed = 0;
    const int32_t* d_seq_steps = nullptr;
    int L = 1;
    int step_value = 0;
    int32_t* sampled = nullptr;      // [B, L] output
};

int lm_head_from_hsel(jot_model* m, int exclude_mask, const int32_t* bump_id, const float* bump_val, float* top1,
                      float* top2, float* sumexp, int32_t* argmax, int M, cudaStream_t st,
                      const HeadSampling* hs = nullptr, int v_lo = 0, int v_hi = 0) {
    const jot_model_config& c = m->cfg;
    if (M <= 0) return JOT_OK;                       // an empty block range has no active rows
    if (M > jot_max_active_rows(m->di->sms)) return JOT_ERR_SHAPE;   // every row block needs a CTA (pair) of its own
    GemmParams p{};
    p.M = m->R_cap; p.N = c.vocab; p.K = c.d_model; p.status = m->ctrl;
    p.d_R = m->ctrl + 1; p.rows = m->rows_out; p.bump_id = bump_id; p.bump_val = bump_val;
    p.mask_col = exclude_mask ? c.mask_id : -1;
    p.partials = m->partials; p.R_pad = m->R_cap;
    p.col_lo = v_lo; p.col_hi = v_hi;                 // (0, 0): the whole vocabulary
    const bool sampling = hs && hs->temperature > 0.f;
    if (sampling) {
        p.inv_temperature = 1.f / hs->temperature; p.sample_seed = hs->seed; p.d_seq_steps = hs->d_seq_steps;
        p.L = hs->L; p.step_value = hs->step_value; p.partials2 = m->partials2;
    }
    // few active rows: the head streams W once and is bandwidth bound -> narrow tiles balance the SMs best;
    // many rows: CTA pairs (256 x 256 tiles) halve the W bytes each SM takes in
    const int mode = (M <= 128) ? 0 : (M <= 256 ? 1 : 2);
    int grid = m->di->sms > 256 ? 256 : m->di->sms;
    int bn = 256;
    {
        ProfScope ps(m, JOT_PROF_LM_HEAD, st);
        if (mode == 0) {
            bn = 128;
            if (sampling) JOT_TRY((launch_gemm_t<128, EPI_STATS_DRAW>(p, m->tm_hsel, m->wlm.m128, grid, st)));
            else JOT_TRY((launch_gemm_t<128, EPI_STATS>(p, m->tm_hsel, m->wlm.m128, grid, st)));
        } else if (mode == 1) {
            if (sampling) JOT_TRY((launch_gemm_t<256, EPI_STATS_DRAW>(p, m->tm_hsel, m->wlm.m256, grid, st)));
            else JOT_TRY((launch_gemm_t<256, EPI_STATS>(p, m->tm_hsel, m->wlm.m256, grid, st)));
        } else {
            grid &= ~1;
            if (sampling) JOT_TRY((launch_pair_t<EPI_STATS_DRAW>(p, m->tm_hsel, m->wlm.m128, grid, st)));
            else JOT_TRY((launch_pair_t<EPI_STATS>(p, m->tm_hsel, m->wlm.m128, grid, st)));
        }
    }
    const int n_vt = ((v_hi > 0 ? v_hi : c.vocab) + bn - 1) / bn - v_lo / bn;     // tiles that touch the slice
    ProfScope ps(m, JOT_PROF_MERGE, st);
    launch_k(merge_stats_kernel, dim3((M + 3) / 4), dim3(128), 0, st, m->partials, m->R_cap, grid, n_vt, mode == 2 ? 1 : 0,
             m->rows_out, m->ctrl + 1, top1, top2, sumexp, argmax, sampling ? m->partials2 : nullptr,
             sampling ? hs->sampled : nullptr);
    return launch_check();
}

// One CTA waits on an mbarrier that nothing ever arms, through the same bounded wait every kernel uses, and
// reports that the wait gave up.  The kernel returns normally: the context stays usable.
__global__ void wait_expiry_kernel(int32_t* status, unsigned long long limit_ns) {
    __shared__ uint64_t never_armed;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&never_armed, 1);
        fence_barrier_init();
    }
    __syncthreads();
    bool ok = true;
    if (threadIdx.x == 0) ok = mbar_wait(&never_armed, 0, &abort_flag, limit_ns);
    __syncthreads();
    if (threadIdx.x == 0) status[0] = ok ? 0 : (abort_flag ? 1 : 2);
}

// copy rows of a [*, d] bf16 matrix selected by `rows` (only r < *d_R)
__global__ void gather_rows_kernel(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int d,
                                   const int32_t* __restrict__ rows, const int32_t* __restrict__ d_R) {
    grid_launch_dependents();
    grid_dependency_wait();
    const int r = blockIdx.x;
    if (r >= *d_R) return;
    const uint4* s = reinterpret_cast<const uint4*>(src + (size_t)rows[r] * d);
    uint4* t = reinterpret_cast<uint4*>(dst + (size_t)r * d);
    for (int i = threadIdx.x; i < d / 8; i += blockDim.x) t[i] = s[i];
}

// public sampling descriptor -> the head's; temperature <= 0 (or no descriptor) means argmax only
int head_sampling_from(const jot_sampling* sp, int32_t* d_sampled, HeadSampling* hs) {
    if (!sp || !(sp->temperature > 0.f)) return JOT_OK;
    if (!d_sampled || sp->step < 0) return JOT_ERR_ARG;
    hs->temperature = sp->temperature;
    hs->seed = sp->seed;
    hs->step_value = sp->step;
    hs->sampled = d_sampled;
    return JOT_OK;
}

int check_step_args(const jot_model* m, const void* tokens, int B, int L, int blk_lo, int blk_hi, const void* bump_id,
                    const void* bump_val, const void* o1, const void* o2, const void* o3, const void* o4) {
    if (!m || !tokens || !o1 || !o2 || !o3 || !o4) return JOT_ERR_ARG;
    if ((bump_id == nullptr) != (bump_val == nullptr)) return JOT_ERR_ARG;
    if (B <= 0 || L <= 0 || blk_lo < 0 || blk_hi > L || blk_lo > blk_hi) return JOT_ERR_ARG;
    if (B > m->max_batch || L > m->max_seq) return JOT_ERR_SHAPE;
    return JOT_OK;
}

// Status word the kernels set: 0 ok; kStatusBadToken: a token id outside the vocabulary (the row was embedded as
// token 0); anything else: a bounded wait expired.
int status_code(int32_t w) { return w == 0 ? JOT_OK : (w == kStatusBadToken ? JOT_ERR_ARG : JOT_ERR_TIMEOUT); }

int read_status(jot_model* m, cudaStream_t st) {
    JOT_CUDA(cudaMemcpyAsync(m->h_pinned, m->ctrl, 4, cudaMemcpyDeviceToHost, st));
    JOT_CUDA(cudaStreamSynchronize(st));
    const int32_t w = m->h_pinned[0];
    if (w == kStatusBadToken) JOT_CUDA(cudaMemsetAsync(m->ctrl, 0, 4, st));     // the caller can fix its input and go on
    return status_code(w);
}

int launch_accept(const AcceptArgs& a, cudaStream_t st, const AcceptParamsInline* inl = nullptr) {
    const size_t smem = accept_smem_bytes(a.L);
    if (smem > 200 * 1024) return JOT_ERR_SHAPE;
    if (inl) {
        if (smem > 48 * 1024)
            JOT_CUDA(cudaFuncSetAttribute(accept_freeze_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        launch_k(accept_freeze_kernel<true>, dim3(a.B), dim3(kAcceptThreads), smem, st, a, *inl);
    } else {
        if (smem > 48 * 1024)
            JOT_CUDA(cudaFuncSetAttribute(accept_freeze_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        launch_k(accept_freeze_kernel<false>, dim3(a.B), dim3(kAcceptThreads), smem, st, a, AcceptParamsNone{});
    }
    return launch_check();
}

bool params_ok(const jot_params* p) {
    if (!p || p->D < 1 || p->D > kMaxD) return false;
    if (p->schedule != JOT_SCHEDULE_FIXED && p->schedule != JOT_SCHEDULE_FRACTIONAL) return false;
    if (p->gate == JOT_GATE_MAXPROB) return p->prob_threshold > 0.f && p->prob_threshold <= 1.f;
    if (p->gate == JOT_GATE_GLOBAL_GAP) return p->gap_threshold == p->gap_threshold;      // anything but NaN
    return p->gate == JOT_GATE_RATIO;
}

}  // namespace

// ---------------------------------------------------------------- exported functions
extern "C" {

const char* jot_status_string(int s) {
    switch (s) {
        case JOT_OK: return "ok";
        case JOT_ERR_ARG: return "invalid argument";
        case JOT_ERR_SHAPE: return "unsupported shape";
        case JOT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case JOT_ERR_CUDA: return "CUDA call failed";
        case JOT_ERR_TIMEOUT: return "bounded device wait expired";
        case JOT_ERR_DEVICE: return "device or driver not supported (needs sm_100 and tensor-map support)";
        case JOT_ERR_LIMIT: return "problem larger than the built-in scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

int jot_last_cuda_error(void) { return g_last_cuda_error; }

int jot_max_active_rows(int n_sms) {
    // more than 256 rows go through CTA pairs (256 rows per pair of SMs), so both forms allow 128 rows per SM
    return n_sms < 2 ? 0 : 128 * (n_sms & ~1);
}

int jot_lm_head_partition(int active_rows, int n_ctas, int vocab_tiles, int pair_mode, int* n_row_blocks, int* n_chunks) {
    if (!n_row_blocks || !n_chunks || active_rows < 0 || n_ctas <= 0 || vocab_tiles <= 0) return JOT_ERR_ARG;
    if (pair_mode) {
        int n_pr = 0;
        stats_partition_pair(active_rows, n_ctas / 2, vocab_tiles, n_row_blocks, &n_pr, n_chunks);
    } else {
        stats_partition(active_rows, n_ctas, vocab_tiles, n_row_blocks, n_chunks);
    }
    return JOT_OK;
}

int jot_set_sync(jot_model* m, int sync) {
    if (!m) return JOT_ERR_ARG;
    m->sync_steps = sync != 0;
    return JOT_OK;
}

int jot_read_status(jot_model* m, void* stream) {
    if (!m) return JOT_ERR_ARG;
    return read_status(m, (cudaStream_t)stream);
}
int64_t jot_launch_count(void) { return g_launches.load(); }

size_t jot_workspace_bytes(const jot_model_config* cfg, int max_batch, int max_seq) {
    if (!config_ok(cfg) || max_batch <= 0 || max_seq <= 0) return 0;
    return make_layout(cfg, max_batch, max_seq).total;
}

int jot_init_model(const jot_model_config* cfg, const jot_weights* w, int max_batch, int max_seq, void* ws,
                   size_t ws_bytes, jot_model** out) {
    if (!cfg || !w || !out) return JOT_ERR_ARG;
    *out = nullptr;
    if (max_batch <= 0 || max_seq <= 0) return JOT_ERR_ARG;
    if (!config_ok(cfg)) return JOT_ERR_SHAPE;
    if (!w->embed || !w->lm_head || !w->final_norm) return JOT_ERR_ARG;
    if (cfg->n_layers > 0 && (!w->attn_norm || !w->wqkv || !w->wo || !w->mlp_norm || !w->w_gate_up || !w->w_down))
        return JOT_ERR_ARG;
    const Layout lay = make_layout(cfg, max_batch, max_seq);
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 1023) || ws_bytes < lay.total) return JOT_ERR_WORKSPACE;
    DeviceInfo* di = nullptr;
    JOT_TRY(device_info(&di));

    jot_model* m = new (std::nothrow) jot_model();
    if (!m) return JOT_ERR_ARG;
    m->cfg = *cfg;
    m->max_batch = max_batch;
    m->max_seq = max_seq;
    m->di_val = *di;
    m->di = &m->di_val;
    m->embed = (const __nv_bfloat16*)w->embed;
    m->lm_head = (const __nv_bfloat16*)w->lm_head;
    m->final_norm = (const __nv_bfloat16*)w->final_norm;
    uint8_t* base = (uint8_t*)ws;
    m->ctrl = (int32_t*)(base + lay.ctrl);
    m->rope_cs = (float2*)(base + lay.rope);
    m->h = (__nv_bfloat16*)(base + lay.h);
    m->a = (__nv_bfloat16*)(base + lay.a);
    m->qkv = (__nv_bfloat16*)(base + lay.qkv);
    m->vt = (__nv_bfloat16*)(base + lay.vt);
    m->attn = (__nv_bfloat16*)(base + lay.attn);
    m->act = (__nv_bfloat16*)(base + lay.act);
    m->hsel = (__nv_bfloat16*)(base + lay.hsel);
    m->rows = (int32_t*)(base + lay.rows);
    m->rows_out = (int32_t*)(base + lay.rows_out);
    m->seq_map = (int32_t*)(base + lay.seq_map);
    m->partials = (float4*)(base + lay.partials);
    m->partials2 = (float2*)(base + lay.partials2);
    m->g_sampled = (int32_t*)(base + lay.sampled);
    m->splitk = (float*)(base + lay.splitk);
    m->R_cap = (int)align_up((size_t)max_batch * max_seq, 128);
    m->canvas = (int32_t*)(base + lay.canvas);
    m->g_top1 = (float*)(base + lay.top1);
    m->g_top2 = (float*)(base + lay.top2);
    m->g_sumexp = (float*)(base + lay.sumexp);
    m->g_argmax = (int32_t*)(base + lay.argmax);
    m->state = (SeqState*)(base + lay.state);
    m->params_dev = (AcceptParamsDev*)(base + lay.params);

    int rc = JOT_OK;
    auto fail = [&](int code) {
        for (cudaEvent_t ev : m->step_done) if (ev) cudaEventDestroy(ev);
        if (m->h_pinned) cudaFreeHost(m->h_pinned);
        delete m;
        return code;
    };
    const int d = cfg->d_model, hd = cfg->head_dim, nq = cfg->n_q_heads, nkv = cfg->n_kv_heads;
    for (int l = 0; l < cfg->n_layers; ++l) {
        if (!w->attn_norm[l] || !w->wqkv[l] || !w->wo[l] || !w->mlp_norm[l] || !w->w_gate_up[l] || !w->w_down[l])
            return fail(JOT_ERR_ARG);
        m->attn_norm.push_back((const __nv_bfloat16*)w->attn_norm[l]);
        m->mlp_norm.push_back((const __nv_bfloat16*)w->mlp_norm[l]);
        WeightMaps wm;
        if ((rc = make_weight_maps(di, &wm, w->wqkv[l], (nq + 2 * nkv) * hd, d, false)) != JOT_OK) return fail(rc);
        m->wqkv.push_back(wm);
        if ((rc = make_weight_maps(di, &wm, w->wo[l], d, nq * hd, false)) != JOT_OK) return fail(rc);
        m->wo.push_back(wm);
        if ((rc = make_weight_maps(di, &wm, w->w_gate_up[l], 2 * cfg->d_ff, d, true)) != JOT_OK) return fail(rc);
        m->wgu.push_back(wm);
        if ((rc = make_weight_maps(di, &wm, w->w_down[l], d, cfg->d_ff, false)) != JOT_OK) return fail(rc);
        m->wdown.push_back(wm);
    }
    if ((rc = make_weight_maps(di, &m->wlm, w->lm_head, cfg->vocab, d, false)) != JOT_OK) return fail(rc);

    // tables: cos/sin of pos * theta^(-2j/hd), evaluated in double on the host once
    std::vector<float2> cs((size_t)max_seq * (hd / 2));
    for (int pos = 0; pos < max_seq; ++pos)
        for (int j = 0; j < hd / 2; ++j) {
            const double ang = (double)pos * std::pow((double)cfg->rope_theta, -2.0 * j / hd);
            cs[(size_t)pos * (hd / 2) + j] = make_float2((float)std::cos(ang), (float)std::sin(ang));
        }
    cudaError_t e = cudaMemcpy(m->rope_cs, cs.data(), cs.size() * sizeof(float2), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(m->ctrl, 0, 1024);
    if (e == cudaSuccess) e = cudaMemset(m->hsel, 0, (size_t)m->R_cap * d * 2);
    if (e == cudaSuccess) e = cudaMemset(m->rows, 0, (size_t)m->R_cap * 4);
    if (e == cudaSuccess) e = cudaMemset(m->rows_out, 0, (size_t)m->R_cap * 4);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&m->step_done[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaHostAlloc((void**)&m->h_pinned, 64 + (size_t)max_batch * sizeof(SeqState), cudaHostAllocDefault);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return fail(JOT_ERR_CUDA);
    }
    *out = m;
    return JOT_OK;
}

int jot_free_model(jot_model* m) {
    if (!m) return JOT_ERR_ARG;
    if (m->h_pinned) cudaFreeHost(m->h_pinned);
    for (cudaEvent_t ev : m->step_done) if (ev) cudaEventDestroy(ev);
    for (cudaEvent_t e : m->ev_pool) cudaEventDestroy(e);
    delete m;
    return JOT_OK;
}

int jot_lm_head_stats(jot_model* m, const void* d_hidden, const int32_t* d_tokens, int B, int L, int blk_lo, int blk_hi,
                      int exclude_mask_token, const int32_t* d_bump_id, const float* d_bump_val, float* d_top1,
                      float* d_top2, float* d_sumexp, int32_t* d_argmax, const jot_sampling* sampling,
                      int32_t* d_sampled, void* stream) {
    return jot_lm_head_stats_slice(m, d_hidden, d_tokens, B, L, blk_lo, blk_hi, exclude_mask_token, d_bump_id, d_bump_val,
                                   0, m ? m->cfg.vocab : 0, d_top1, d_top2, d_sumexp, d_argmax, sampling, d_sampled, stream);
}

int jot_merge_stats(int n, const float* a_top1, const float* a_top2, const float* a_sumexp, const int32_t* a_argmax,
                    const float* b_top1, const float* b_top2, const float* b_sumexp, const int32_t* b_argmax,
                    float* o_top1, float* o_top2, float* o_sumexp, int32_t* o_argmax, void* stream) {
    if (n < 0 || !a_top1 || !a_top2 || !a_sumexp || !a_argmax || !b_top1 || !b_top2 || !b_sumexp || !b_argmax || !o_top1 ||
        !o_top2 || !o_sumexp || !o_argmax)
        return JOT_ERR_ARG;
    if (n == 0) return JOT_OK;
    launch_k(merge_stat_arrays_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, (cudaStream_t)stream, n, a_top1, a_top2,
             a_sumexp, a_argmax, b_top1, b_top2, b_sumexp, b_argmax, o_top1, o_top2, o_sumexp, o_argmax);
    return launch_check();
}

int jot_lm_head_stats_slice(jot_model* m, const void* d_hidden, const int32_t* d_tokens, int B, int L, int blk_lo,
                            int blk_hi, int exclude_mask_token, const int32_t* d_bump_id, const float* d_bump_val,
                            int v_lo, int v_hi, float* d_top1, float* d_top2, float* d_sumexp, int32_t* d_argmax,
                            const jot_sampling* sampling, int32_t* d_sampled, void* stream) {
    JOT_TRY(check_step_args(m, d_tokens, B, L, blk_lo, blk_hi, d_bump_id, d_bump_val, d_top1, d_top2, d_sumexp, d_argmax));
    if (!d_hidden) return JOT_ERR_ARG;
    if (v_lo < 0 || v_hi > m->cfg.vocab || v_lo >= v_hi) return JOT_ERR_ARG;
    const bool whole = v_lo == 0 && v_hi == m->cfg.vocab;
    if (!whole && sampling && sampling->temperature > 0.f) return JOT_ERR_ARG;   // a draw needs the whole vocabulary
    HeadSampling hs;
    JOT_TRY(head_sampling_from(sampling, d_sampled, &hs));
    cudaStream_t st = (cudaStream_t)stream;
    JOT_TRY(encode_activation_maps(m, B, L));
    {
        ProfScope ps(m, JOT_PROF_ROWS, st);
        launch_k(build_rows_kernel, dim3(1), dim3(1024), 0, st, d_tokens, B, L, m->cfg.mask_id, blk_lo, blk_hi, nullptr, 0, 0, 0, nullptr, m->rows, m->rows_out,
                                              m->ctrl + 1, L, 0);
        JOT_TRY(launch_check());
        launch_k(gather_rows_kernel, dim3(B * L), dim3(128), 0, st, (const __nv_bfloat16*)d_hidden, m->hsel, m->cfg.d_model, m->rows,
                                                  m->ctrl + 1);
        JOT_TRY(launch_check());
    }
    JOT_TRY(lm_head_from_hsel(m, exclude_mask_token, d_bump_id, d_bump_val, d_top1, d_top2, d_sumexp, d_argmax,
                              B * (blk_hi - blk_lo), st, &hs, whole ? 0 : v_lo, whole ? 0 : v_hi));
    return m->sync_steps ? read_status(m, st) : JOT_OK;
}

namespace {
int denoise_step_impl(jot_model* m, const int32_t* d_tokens, int B, int L, int blk_lo, int blk_hi, int exclude_mask_token,
                      const int32_t* d_bump_id, const float* d_bump_val, float* d_top1, float* d_top2, float* d_sumexp,
                      int32_t* d_argmax, const jot_sampling* sampling, int32_t* d_sampled, void* stream,
                      const FwdSpan* span) {
    JOT_TRY(check_step_args(m, d_tokens, B, L, blk_lo, blk_hi, d_bump_id, d_bump_val, d_top1, d_top2, d_sumexp, d_argmax));
    HeadSampling hs;
    JOT_TRY(head_sampling_from(sampling, d_sampled, &hs));
    cudaStream_t st = (cudaStream_t)stream;
    const int Lr = span ? span->Lr : L, pos0 = span ? span->pos0 : 0;
    JOT_TRY(forward_body(m, d_tokens, B, L, st, nullptr, span));
    {
        ProfScope ps(m, JOT_PROF_ROWS, st);
        launch_k(build_rows_kernel, dim3(1), dim3(1024), 0, st, d_tokens, B, L, m->cfg.mask_id, blk_lo, blk_hi, nullptr, 0, 0, 0, nullptr, m->rows, m->rows_out,
                                              m->ctrl + 1, Lr, pos0);
        JOT_TRY(launch_check());
        launch_k(rmsnorm_kernel, dim3(std::max(1, B * (blk_hi - blk_lo))), dim3(256), 0, st, m->h, m->final_norm, m->hsel, m->cfg.d_model, m->cfg.rms_eps, m->rows,
                                              m->ctrl + 1);
        JOT_TRY(launch_check());
    }
    JOT_TRY(lm_head_from_hsel(m, exclude_mask_token, d_bump_id, d_bump_val, d_top1, d_top2, d_sumexp, d_argmax,
                              B * (blk_hi - blk_lo), st, &hs));
    return m->sync_steps ? read_status(m, st) : JOT_OK;
}
}  // namespace

int jot_denoise_step(jot_model* m, const int32_t* d_tokens, int B, int L, int blk_lo, int blk_hi, int exclude_mask_token,
                     const int32_t* d_bump_id, const float* d_bump_val, float* d_top1, float* d_top2, float* d_sumexp,
                     int32_t* d_argmax, const jot_sampling* sampling, int32_t* d_sampled, void* stream) {
    return denoise_step_impl(m, d_tokens, B, L, blk_lo, blk_hi, exclude_mask_token, d_bump_id, d_bump_val, d_top1, d_top2,
                             d_sumexp, d_argmax, sampling, d_sampled, stream, nullptr);
}

size_t jot_kv_cache_bytes(const jot_model_config* cfg, int max_batch, int max_seq) {
    if (!config_ok(cfg) || max_batch <= 0 || max_seq <= 0) return 0;
    return (size_t)cfg->n_layers * kv_layer_bytes(cfg, max_batch, max_seq, nullptr) + 1024;
}

int jot_attach_kv_cache(jot_model* m, void* d_cache, size_t bytes) {
    if (!m) return JOT_ERR_ARG;
    m->kv_map_B = m->kv_map_L = m->kv_valid_B = m->kv_valid_L = -1;
    m->kv_base = nullptr;
    m->kv_bytes = 0;
    if (!d_cache) return JOT_OK;                                   // detach
    if (reinterpret_cast<uintptr_t>(d_cache) & 1023) return JOT_ERR_ARG;
    if (bytes < jot_kv_cache_bytes(&m->cfg, m->max_batch, m->max_seq)) return JOT_ERR_WORKSPACE;
    size_t vt_off = 0;
    const size_t per_layer = kv_layer_bytes(&m->cfg, m->max_batch, m->max_seq, &vt_off);
    const int n = m->cfg.n_layers;
    m->kv_qkv.resize(n); m->kv_vt.resize(n); m->kv_tm_qkv3.resize(n); m->kv_tm_vt.resize(n);
    for (int l = 0; l < n; ++l) {
        uint8_t* base = (uint8_t*)d_cache + (size_t)l * per_layer;
        m->kv_qkv[l] = (__nv_bfloat16*)base;
        m->kv_vt[l] = (__nv_bfloat16*)(base + vt_off);
    }
    m->kv_base = (uint8_t*)d_cache;
    m->kv_bytes = bytes;
    return JOT_OK;
}

int jot_denoise_step_cached(jot_model* m, const int32_t* d_tokens, int B, int L, int blk_lo, int blk_hi, int refresh,
                            int exclude_mask_token, const int32_t* d_bump_id, const float* d_bump_val, float* d_top1,
                            float* d_top2, float* d_sumexp, int32_t* d_argmax, const jot_sampling* sampling,
                            int32_t* d_sampled, void* stream) {
    if (!m || !m->kv_base) return JOT_ERR_ARG;
    if (blk_lo >= blk_hi) return JOT_ERR_ARG;
    if (!refresh && (m->kv_valid_B != B || m->kv_valid_L != L)) return JOT_ERR_ARG;     // nothing cached for this canvas
    const FwdSpan span = refresh ? FwdSpan{L, 0, true} : FwdSpan{blk_hi - blk_lo, blk_lo, true};
    const int rc = denoise_step_impl(m, d_tokens, B, L, blk_lo, blk_hi, exclude_mask_token, d_bump_id, d_bump_val, d_top1,
                                     d_top2, d_sumexp, d_argmax, sampling, d_sampled, stream, &span);
    if (rc == JOT_OK && refresh) { m->kv_valid_B = B; m->kv_valid_L = L; }
    return rc;
}

int jot_accept_freeze(const jot_params* params, int per_seq_params, int32_t mask_id, int32_t* d_tokens, int B, int L,
                      int blk_lo, int blk_hi, int k_transfer, const float* d_top1, const float* d_top2,
                      const float* d_sumexp, const int32_t* d_argmax, int32_t* d_n_masked, uint8_t* d_exit_reason,
                      int16_t* d_exit_step, int step_index, void* stream) {
    if (!params || !d_tokens || !d_top1 || !d_top2 || !d_sumexp || !d_argmax) return JOT_ERR_ARG;
    if (B <= 0 || L <= 0 || blk_lo < 0 || blk_hi > L || blk_lo > blk_hi || k_transfer < 0) return JOT_ERR_ARG;
    const int n_par = per_seq_params ? B : 1;
    if (n_par > kAcceptInlineParams) return JOT_ERR_SHAPE;       // B parameter sets travel as kernel arguments
    for (int i = 0; i < n_par; ++i)
        if (!params_ok(params + i)) return JOT_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    static_assert(sizeof(AcceptParamsDev) == sizeof(jot_params), "parameter struct layouts must agree");
    AcceptArgs a{};
    AcceptParamsInline inl{};
    memcpy(inl.p, params, (size_t)n_par * sizeof(jot_params));
    a.uniform = inl.p[0];
    a.params = nullptr;
    a.per_seq_params = per_seq_params ? 1 : 0;
    a.mask_id = mask_id; a.tokens = d_tokens; a.B = B; a.L = L;
    a.blk_lo = blk_lo; a.blk_hi = blk_hi; a.k_transfer = k_transfer;
    a.top1 = d_top1; a.top2 = d_top2; a.sumexp = d_sumexp; a.argmax = d_argmax;
    a.n_masked = d_n_masked; a.exit_reason = d_exit_reason; a.exit_step = d_exit_step; a.step_index = step_index;
    a.state = nullptr;
    JOT_TRY(launch_accept(a, st, per_seq_params ? &inl : nullptr));
    return JOT_OK;
}

int jot_generate(jot_model* m, const jot_params* params, int per_seq_params, const jot_gen_config* gen,
                 const int32_t* d_prompt, int B, int P, const int32_t* d_bump_id, const float* d_bump_val,
                 int32_t* d_out_tokens, int32_t* h_steps_used, int32_t* h_forward_passes, const jot_trace* trace,
                 void* stream) {
    if (!m || !params || !gen || !d_out_tokens || !h_steps_used) return JOT_ERR_ARG;
    if ((d_bump_id == nullptr) != (d_bump_val == nullptr)) return JOT_ERR_ARG;
    if (B <= 0 || P < 0 || gen->gen_len <= 0 || gen->steps <= 0 || gen->block_len <= 0) return JOT_ERR_ARG;
    if (P > 0 && !d_prompt) return JOT_ERR_ARG;
    if (gen->gen_len % gen->block_len) return JOT_ERR_ARG;
    const int nb = gen->gen_len / gen->block_len;
    if (gen->steps % nb) return JOT_ERR_ARG;
    const int Tb = gen->steps / nb, L = P + gen->gen_len;
    if (B > m->max_batch || L > m->max_seq) return JOT_ERR_SHAPE;
    const int n_par = per_seq_params ? B : 1;
    for (int i = 0; i < n_par; ++i)
        if (!params_ok(params + i)) return JOT_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    static_assert(sizeof(AcceptParamsDev) == sizeof(jot_params), "parameter struct layouts must agree");
    static_assert(sizeof(SeqState) == 16 && offsetof(SeqState, steps_used) == 8, "the head reads steps_used at int 2 of 4");
    JOT_CUDA(cudaMemcpyAsync(m->params_dev, params, (size_t)n_par * sizeof(jot_params), cudaMemcpyHostToDevice, st));
    launch_k(init_canvas_kernel, dim3((B * L + 255) / 256), dim3(256), 0, st, d_prompt, m->canvas, B, P, gen->gen_len, m->cfg.mask_id,
                                                           m->state);
    JOT_TRY(launch_check());
    if (trace) {                                     // positions and steps that never occur read as zero
        if (trace->d_exit_step) JOT_CUDA(cudaMemsetAsync(trace->d_exit_step, 0, (size_t)B * L * sizeof(int16_t), st));
        if (trace->d_exit_reason) JOT_CUDA(cudaMemsetAsync(trace->d_exit_reason, 0, (size_t)B * L, st));
        if (trace->d_mean_ratio) JOT_CUDA(cudaMemsetAsync(trace->d_mean_ratio, 0, (size_t)gen->steps * B * sizeof(float), st));
        if (trace->d_n_candidates)
            JOT_CUDA(cudaMemsetAsync(trace->d_n_candidates, 0, (size_t)gen->steps * B * sizeof(int32_t), st));
    }
    // The host runs one step ahead of what it knows: step `it` is enqueued before the outcome of step it-1 has
    // been read, so the GPU never idles while the host looks at the loop condition.  A step enqueued after the
    // last sequence finished finds nothing masked and changes nothing; it is not counted.
    int passes = 0;
    int B_act = B;                                   // upper bound on the sequences that still have work
    const bool compact = gen->compact_finished != 0;
    auto outcome = [&](int slot, bool* finished) -> int {      // wait for a step's control words
        JOT_CUDA(cudaEventSynchronize(m->step_done[slot]));
        const int32_t* w = m->h_pinned + 4 * slot;
        if (w[0]) {
            if (w[0] == kStatusBadToken) cudaMemsetAsync(m->ctrl, 0, 4, st);
            return status_code(w[0]);
        }
        *finished = w[2] == 0;
        if (!*finished) B_act = w[2];
        return JOT_OK;
    };
    // sampling-based finalisation: the step index is read from the per-sequence state on the device, so a
    // captured step can be replayed unchanged
    const bool sampling = gen->temperature > 0.f;
    HeadSampling hs;
    if (sampling) {
        hs.temperature = gen->temperature;
        hs.seed = ((unsigned long long)gen->seed_hi << 32) | gen->seed_lo;
        hs.d_seq_steps = reinterpret_cast<const int32_t*>(m->state) + 2;      // SeqState::steps_used
        hs.L = L;
        hs.sampled = m->g_sampled;
    }
    if (gen->kv_cache) {
        // Block-wise KV cache: every sequence works on the same block.  The first step of a block runs the whole
        // canvas and leaves every layer's keys and values in the cache; the block's other steps run only the
        // block's rows against it.  The host reads the block's outcome after every step (what runs next depends
        // on it), so this loop is not pipelined.
        if (!m->kv_base) return JOT_ERR_ARG;
        const int Lb = gen->block_len;
        int n_passes = 0;
        for (int blk = 0; blk < nb; ++blk) {
            const int lo = P + blk * Lb, hi = lo + Lb;
            for (int s = 0; s < Tb; ++s) {
                JOT_CUDA(cudaMemsetAsync(m->ctrl + 2, 0, 4, st));
                const FwdSpan span = (s == 0) ? FwdSpan{L, 0, true} : FwdSpan{Lb, lo, true};
                JOT_TRY(forward_body(m, m->canvas, B, L, st, nullptr, &span));
                {
                    ProfScope ps(m, JOT_PROF_ROWS, st);
                    launch_k(build_rows_kernel, dim3(1), dim3(1024), 0, st, m->canvas, B, L, m->cfg.mask_id, lo, hi, nullptr, 0,
                             0, 0, nullptr, m->rows, m->rows_out, m->ctrl + 1, span.Lr, span.pos0);
                    JOT_TRY(launch_check());
                    launch_k(rmsnorm_kernel, dim3(B * Lb), dim3(256), 0, st, m->h, m->final_norm, m->hsel, m->cfg.d_model,
                             m->cfg.rms_eps, m->rows, m->ctrl + 1);
                    JOT_TRY(launch_check());
                }
                JOT_TRY(lm_head_from_hsel(m, gen->exclude_mask_token, d_bump_id, d_bump_val, m->g_top1, m->g_top2,
                                          m->g_sumexp, m->g_argmax, B * Lb, st, &hs));
                AcceptArgs a{};
                a.params = m->params_dev; a.per_seq_params = per_seq_params ? 1 : 0;
                a.mask_id = m->cfg.mask_id; a.tokens = m->canvas; a.B = B; a.L = L;
                a.top1 = m->g_top1; a.top2 = m->g_top2; a.sumexp = m->g_sumexp;
                a.argmax = sampling ? m->g_sampled : m->g_argmax;
                a.state = m->state; a.lockstep = 1; a.lockstep_s = s; a.steps_per_block = Tb; a.blk_lo = lo; a.blk_hi = hi;
                a.k_transfer = Lb / Tb + (s < Lb % Tb ? 1 : 0);
                a.n_unfinished = m->ctrl + 2;
                if (trace) {
                    a.exit_step = trace->d_exit_step; a.exit_reason = trace->d_exit_reason;
                    a.mean_ratio = trace->d_mean_ratio; a.n_candidates = trace->d_n_candidates;
                }
                {
                    ProfScope ps(m, JOT_PROF_ACCEPT, st);
                    JOT_TRY(launch_accept(a, st));
                }
                JOT_CUDA(cudaMemcpyAsync(m->h_pinned, m->ctrl, 16, cudaMemcpyDeviceToHost, st));
                JOT_CUDA(cudaStreamSynchronize(st));
                if (m->h_pinned[0]) {
                    const int32_t w0 = m->h_pinned[0];
                    if (w0 == kStatusBadToken) cudaMemsetAsync(m->ctrl, 0, 4, st);
                    return status_code(w0);
                }
                ++n_passes;
                if (m->h_pinned[2] == 0) break;              // no sequence has a masked position left in this block
            }
        }
        m->kv_valid_B = m->kv_valid_L = -1;                  // the cache belongs to a canvas that is finished
        JOT_CUDA(cudaMemcpyAsync(d_out_tokens, m->canvas, (size_t)B * L * 4, cudaMemcpyDeviceToDevice, st));
        SeqState* hstate = reinterpret_cast<SeqState*>(m->h_pinned + 16);
        JOT_CUDA(cudaMemcpyAsync(hstate, m->state, (size_t)B * sizeof(SeqState), cudaMemcpyDeviceToHost, st));
        JOT_CUDA(cudaStreamSynchronize(st));
        for (int b = 0; b < B; ++b) h_steps_used[b] = hstate[b].steps_used;
        if (h_forward_passes) *h_forward_passes = n_passes;
        return JOT_OK;
    }
    // everything one step enqueues, ending with the copy of the control words to the pinned slot it & 1
    auto enqueue_step = [&](int it, int Bf, const int32_t* seq_map) -> int {
        JOT_CUDA(cudaMemsetAsync(m->ctrl + 2, 0, 4, st));
        if (seq_map) {
            // finished sequences drop out of the forward pass: the batch is compacted to the live ones
            launch_k(build_seq_map_kernel, dim3(1), dim3(32), 0, st, m->state, B, nb, m->seq_map, m->ctrl + 3);
            JOT_TRY(launch_check());
        }
        JOT_TRY(forward_body(m, m->canvas, Bf, L, st, seq_map));
        {
            ProfScope ps(m, JOT_PROF_ROWS, st);
            launch_k(build_rows_kernel, dim3(1), dim3(1024), 0, st, m->canvas, Bf, L, m->cfg.mask_id, 0, 0, m->state, P,
                     gen->block_len, nb, seq_map, m->rows, m->rows_out, m->ctrl + 1, L, 0);
            JOT_TRY(launch_check());
            launch_k(rmsnorm_kernel, dim3(Bf * L), dim3(256), 0, st, m->h, m->final_norm, m->hsel, m->cfg.d_model,
                     m->cfg.rms_eps, m->rows, m->ctrl + 1);
            JOT_TRY(launch_check());
        }
        JOT_TRY(lm_head_from_hsel(m, gen->exclude_mask_token, d_bump_id, d_bump_val, m->g_top1, m->g_top2, m->g_sumexp,
                                  m->g_argmax, Bf * gen->block_len, st, &hs));
        AcceptArgs a{};
        a.params = m->params_dev; a.per_seq_params = per_seq_params ? 1 : 0;
        a.mask_id = m->cfg.mask_id; a.tokens = m->canvas; a.B = B; a.L = L;
        a.top1 = m->g_top1; a.top2 = m->g_top2; a.sumexp = m->g_sumexp;
        a.argmax = sampling ? m->g_sampled : m->g_argmax;       // the token a finalised position receives
        a.step_index = it + 1;                       // only reaches the optional exit-step output, unused here
        a.state = m->state; a.P = P; a.block_len = gen->block_len; a.n_blocks = nb; a.steps_per_block = Tb;
        a.n_unfinished = m->ctrl + 2;
        if (trace) {
            a.exit_step = trace->d_exit_step; a.exit_reason = trace->d_exit_reason;
            a.mean_ratio = trace->d_mean_ratio; a.n_candidates = trace->d_n_candidates;
        }
        {
            ProfScope ps(m, JOT_PROF_ACCEPT, st);
            JOT_TRY(launch_accept(a, st));
        }
        JOT_CUDA(cudaMemcpyAsync(m->h_pinned + 4 * (it & 1), m->ctrl, 16, cudaMemcpyDeviceToHost, st));
        return JOT_OK;
    };
    // With use_cuda_graph the step is captured once per (batch size after compaction, pinned slot) and replayed:
    // the step's few dozen launches become one graph launch, which is what a small model's step time consists of.
    struct StepGraph { int Bf, slot; cudaGraphExec_t exec; int64_t launches; };
    std::vector<StepGraph> graphs;
    auto release_graphs = [&]() {
        for (auto& g : graphs) cudaGraphExecDestroy(g.exec);
        graphs.clear();
    };
    const bool want_graph = gen->use_cuda_graph != 0 && !m->profiling;
    bool graph_ok = want_graph;
    bool finished = false;
    int rc = JOT_OK;
    for (int it = 0; it < gen->steps && !finished; ++it) {
        const int32_t* seq_map = (compact && B_act < B) ? m->seq_map : nullptr;
        const int Bf = seq_map ? B_act : B;
        bool launched = false;
        if (graph_ok && it >= 1) {                   // step 0 runs eagerly (one-time attribute and map set-up)
            StepGraph* g = nullptr;
            for (auto& c : graphs) if (c.Bf == Bf && c.slot == (it & 1)) g = &c;
            if (!g) {
                cudaGraph_t graph = nullptr;
                const int64_t before = g_launches.load();
                if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
                    const int erc = enqueue_step(it, Bf, seq_map);
                    const cudaError_t ce = cudaStreamEndCapture(st, &graph);
                    cudaGraphExec_t exec = nullptr;
                    if (erc == JOT_OK && ce == cudaSuccess && graph &&
                        cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess) {
                        graphs.push_back({Bf, it & 1, exec, g_launches.load() - before});
                        g = &graphs.back();
                    }
                    if (graph) cudaGraphDestroy(graph);
                }
                g_launches.store(before);            // captured launches are counted when the graph runs
                if (!g) {                            // capture is unavailable: go on with plain launches
                    cudaGetLastError();
                    graph_ok = false;
                }
            }
            if (g) {
                if (cudaGraphLaunch(g->exec, st) != cudaSuccess) { rc = JOT_ERR_CUDA; g_last_cuda_error = (int)cudaGetLastError(); break; }
                g_launches.fetch_add(g->launches);
                launched = true;
            }
        }
        if (!launched && (rc = enqueue_step(it, Bf, seq_map)) != JOT_OK) break;
        if (cudaEventRecord(m->step_done[it & 1], st) != cudaSuccess) { rc = JOT_ERR_CUDA; break; }
        if (it >= 1) {
            if ((rc = outcome((it - 1) & 1, &finished)) != JOT_OK) break;   // step it-1; step `it` is already in flight
            if (finished) break;                                             // ... and was a no-op
        }
        ++passes;
        if (it == gen->steps - 1 && (rc = outcome(it & 1, &finished)) != JOT_OK) break;
    }
    if (rc != JOT_OK) {
        cudaStreamSynchronize(st);
        release_graphs();
        return rc;
    }
    JOT_CUDA(cudaMemcpyAsync(d_out_tokens, m->canvas, (size_t)B * L * 4, cudaMemcpyDeviceToDevice, st));
    SeqState* host_state = reinterpret_cast<SeqState*>(m->h_pinned + 16);
    JOT_CUDA(cudaMemcpyAsync(host_state, m->state, (size_t)B * sizeof(SeqState), cudaMemcpyDeviceToHost, st));
    JOT_CUDA(cudaStreamSynchronize(st));
    release_graphs();
    for (int b = 0; b < B; ++b) h_steps_used[b] = host_state[b].steps_used;
    if (h_forward_passes) *h_forward_passes = passes;
    return JOT_OK;
}

int jot_selftest_wait_expiry(int32_t* d_status, uint64_t limit_ns, void* stream) {
    if (!d_status || limit_ns == 0 || limit_ns > 5000000000ull) return JOT_ERR_ARG;
    wait_expiry_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(d_status, (unsigned long long)limit_ns);
    return launch_check();
}

int jot_profile(jot_model* m, int enable) {
    if (!m) return JOT_ERR_ARG;
    m->profiling = enable != 0;
    m->spans.clear();
    m->ev_used = 0;
    for (int i = 0; i < JOT_PROF_CLASSES; ++i) { m->prof_ms[i] = 0; m->prof_n[i] = 0; }
    return JOT_OK;
}

int jot_profile_read(jot_model* m, double* ms, int64_t* launches, int n_classes) {
    if (!m || !ms || !launches || n_classes < JOT_PROF_CLASSES) return JOT_ERR_ARG;
    for (const auto& sp : m->spans) {
        JOT_CUDA(cudaEventSynchronize(sp.b));
        float t = 0.f;
        JOT_CUDA(cudaEventElapsedTime(&t, sp.a, sp.b));
        m->prof_ms[sp.cls] += t;
        m->prof_n[sp.cls] += 1;
    }
    m->spans.clear();
    m->ev_used = 0;
    for (int i = 0; i < JOT_PROF_CLASSES; ++i) { ms[i] = m->prof_ms[i]; launches[i] = m->prof_n[i]; }
    return JOT_OK;
}

int jot_gemm_bf16(const void* d_A, const void* d_W, const void* d_residual, void* d_C, int M, int N, int K,
                  void* d_scratch, size_t scratch_bytes, int32_t* d_status, void* stream) {
    if (!d_A || !d_W || !d_C) return JOT_ERR_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return JOT_ERR_ARG;
    if (N % 8 || K % 8) return JOT_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(d_A) | reinterpret_cast<uintptr_t>(d_W) | reinterpret_cast<uintptr_t>(d_C) |
         reinterpret_cast<uintptr_t>(d_residual)) & 15)
        return JOT_ERR_ARG;
    DeviceInfo* di = nullptr;
    JOT_TRY(device_info(&di));
    CUtensorMap tmA;
    WeightMaps wm;
    JOT_TRY(make_map_2d(di, &tmA, d_A, M, K, K, 128));
    JOT_TRY(make_weight_maps(di, &wm, d_W, N, K, false));
    GemmParams p{};
    p.M = M; p.N = N; p.K = K; p.C = (__nv_bfloat16*)d_C; p.residual = (const __nv_bfloat16*)d_residual; p.ldc = N;
    p.status = d_status;
    if (d_scratch && (reinterpret_cast<uintptr_t>(d_scratch) & 15)) return JOT_ERR_ARG;
    SlabMaps tmX;
    const bool slab = M <= kSlabMaxTokens && !d_scratch;      // with scratch: K ranges through global memory
    if (slab) JOT_TRY(make_slab_maps(di, &tmX, d_A, M, K, K));
    return run_gemm(di, tmA, wm, EPI_STORE, p, (cudaStream_t)stream, (float*)d_scratch, d_scratch ? scratch_bytes : 0,
                    nullptr, slab ? &tmX : nullptr);
}

}  // extern "C"

// ---------------------------------------------------------------- projection without any allocation
// Split-K needs room for its fp32 partial sums.  Here that room is a fixed array that is part of the
// library image: every GPU that loads the library carries these 16 MiB until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[JOT_NOALLOC_SCRATCH_BYTES];

namespace {
std::mutex g_noalloc_mu;
float* g_noalloc_ptr[64] = {};

// The array's name is only a handle on the host side; its device address has to be asked for, once
// per device, with that device current.
int noalloc_scratch_address(float** out) {
    int dev = 0;
    JOT_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return JOT_ERR_DEVICE;
    std::lock_guard<std::mutex> lock(g_noalloc_mu);
    if (!g_noalloc_ptr[dev]) {
        void* ptr = nullptr;
        JOT_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        if (!ptr) return JOT_ERR_DEVICE;
        g_noalloc_ptr[dev] = static_cast<float*>(ptr);
    }
    *out = g_noalloc_ptr[dev];
    return JOT_OK;
}
}  // namespace

#ifdef JOT_ATTN_TRACE
extern "C" int jot_debug_attn_trace(long long* h_out, int n_words, int reset) {
    if (reset) {
        static long long zeros[256 * 16] = {};
        return cudaMemcpyToSymbol(g_attn_trace, zeros, sizeof(zeros)) == cudaSuccess ? 0 : -4;
    }
    return cudaMemcpyFromSymbol(h_out, g_attn_trace, (size_t)n_words * 8) == cudaSuccess ? 0 : -4;
}
#endif

#ifdef JOT_SLAB_TRACE
extern "C" int jot_debug_slab_trace(unsigned long long* h_out, int n_words) {
    return cudaMemcpyFromSymbol(h_out, g_slab_trace, (size_t)n_words * 8) == cudaSuccess ? 0 : -4;
}
#endif

extern "C" int jot_gemm_bf16_noalloc(const void* d_A, const void* d_W, const void* d_residual, void* d_C, int M, int N,
                                     int K, int32_t* d_status, void* stream) {
    if (!d_A || !d_W || !d_C) return JOT_ERR_ARG;
    if (M <= 0 || N <= 0 || K <= 0) return JOT_ERR_ARG;
    if (N % 8 || K % 8) return JOT_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(d_A) | reinterpret_cast<uintptr_t>(d_W) | reinterpret_cast<uintptr_t>(d_C) |
         reinterpret_cast<uintptr_t>(d_residual)) & 15)
        return JOT_ERR_ARG;
    // room for four K ranges of the whole output, whatever split the kernel then picks
    if ((size_t)M * (size_t)N * 4 * sizeof(float) > (size_t)JOT_NOALLOC_SCRATCH_BYTES) return JOT_ERR_LIMIT;
    DeviceInfo* di = nullptr;
    JOT_TRY(device_info(&di));
    float* scratch = nullptr;
    JOT_TRY(noalloc_scratch_address(&scratch));
    CUtensorMap tmA;
    WeightMaps wm;
    JOT_TRY(make_map_2d(di, &tmA, d_A, M, K, K, 128));
    JOT_TRY(make_weight_maps(di, &wm, d_W, N, K, false));
    GemmParams p{};
    p.M = M; p.N = N; p.K = K; p.C = (__nv_bfloat16*)d_C; p.residual = (const __nv_bfloat16*)d_residual; p.ldc = N;
    p.status = d_status;
    return run_gemm(di, tmA, wm, EPI_STORE, p, (cudaStream_t)stream, scratch, (size_t)JOT_NOALLOC_SCRATCH_BYTES);
}
