// Host side of libowlverify: argument checks, workspace, kernel launches.  C ABI in owlverify.h.
#include "../../include/owlverify.h"

#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <cmath>
#include <mutex>
#include <new>

#include "accept.cuh"
#include "combine.cuh"
#include "gemm_umma_pair.cuh"
#include "owl_common.cuh"
#include "spec_loop.cuh"
#include "verify_attn_umma.cuh"

using namespace owl;

constexpr int kMapCacheEntries = 8;

struct owl_ctx {
    int device = 0;
    int sm_count = 0;
    owl_dims max_dims{};
    int num_ctas = 0;
    int rows_per_slot = 0;
    long long slots = 0;
    float* part_o = nullptr;
    float* part_lse = nullptr;
    int32_t* status = nullptr;
    unsigned long long* selftest_ns = nullptr;
    int32_t* seq_bad = nullptr;
    long long* sched_seq_begin = nullptr;
    SchedHeader* sched_header = nullptr;
    unsigned long long* part_keys = nullptr;
    unsigned long long* lm_keys = nullptr;      // two sets of one arg-max key per row for the LM-head product's epilogue
    uint32_t lm_epoch = 0;                      // calls launched so far: set (lm_epoch & 1) is in use, the other one clean
    unsigned int* seq_counter = nullptr;
    uint32_t accept_epoch = 0;
    long long part_keys_len = 0;
    // tensor maps over the callers' K and V caches: a few most recently used (cache pointers, geometry) pairs
    // are kept, so that a caller rotating over several caches does not pay two encodes per call
    EncodeTiledFn encode = nullptr;
    struct MapEntry {
        CUtensorMap kmap{}, vmap{};
        const void* k = nullptr;
        const void* v = nullptr;
        int pages = 0, heads = 0, page_size = 0;
        bool fp16 = false;
        uint64_t used = 0;
    } maps[kMapCacheEntries];
    uint64_t map_clock = 0;
    int32_t epoch = 0;
    int64_t launches = 0;
    bool profiling = false;
    cudaEvent_t ev[6] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
    bool ev_attn_valid = false, ev_accept_valid = false;
    char err[256] = {0};
    // device staging of owl_verify_step_host (grown on demand)
    struct Staging { void* p = nullptr; size_t cap = 0; } stg[16];
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() { if (switched) cudaSetDevice(prev); }
};

int cuda_fail(owl_ctx* ctx, cudaError_t e, const char* what) {
    if (ctx) snprintf(ctx->err, sizeof ctx->err, "%s: %s", what, cudaGetErrorString(e));
    return OWL_ERR_CUDA;
}

// Launch `kernel(arg)` so that it may be scheduled while the kernel before it in the stream is still running
// (programmatic dependent launch); the kernel itself waits (griddepcontrol.wait) before it reads anything.
template <typename... Args>
cudaError_t launch_dependent_smem(void (*kernel)(Args...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, const Args&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}
template <typename... Args>
cudaError_t launch_dependent(void (*kernel)(Args...), dim3 grid, dim3 block, cudaStream_t stream, const Args&... args) {
    return launch_dependent_smem(kernel, grid, block, 0, stream, args...);
}

// The attention kernel's instances: [more than 32 sequences][units above 128 rows][logits scan fused in], bf16;
// and the fp16 ones (attention only): [more than 32 sequences][units above 128 rows]
using UmmaKernel = void (*)(AttnParams, CUtensorMap, CUtensorMap, AcceptParams);
UmmaKernel umma_kernel(bool many, bool wide, bool fused, bool fp16) {
    using namespace umma_path;
    static const UmmaKernel table[2][2][2] = {
        {{verify_attn_umma_kernel<false, false, false, false>, verify_attn_umma_kernel<false, false, true, false>},
         {verify_attn_umma_kernel<false, true, false, false>, verify_attn_umma_kernel<false, true, true, false>}},
        {{verify_attn_umma_kernel<true, false, false, false>, verify_attn_umma_kernel<true, false, true, false>},
         {verify_attn_umma_kernel<true, true, false, false>, verify_attn_umma_kernel<true, true, true, false>}}};
    static const UmmaKernel table16[2][2] = {
        {verify_attn_umma_kernel<false, false, false, true>, verify_attn_umma_kernel<false, true, false, true>},
        {verify_attn_umma_kernel<true, false, false, true>, verify_attn_umma_kernel<true, true, false, true>}};
    return fp16 ? table16[many][wide] : table[many][wide][fused];
}
bool set_umma_smem_attr() {
    bool ok = true;
    for (int i = 0; i < 8; ++i)
        ok = ok && cudaFuncSetAttribute(umma_kernel(i & 4, i & 2, i & 1, false), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        umma_path::kSmemBytes) == cudaSuccess;
    for (int i = 0; i < 4; ++i)
        ok = ok && cudaFuncSetAttribute(umma_kernel(i & 2, i & 1, false, true), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        umma_path::kSmemBytes) == cudaSuccess;
    return ok;
}

int log2_exact(int v) {
    int s = 0;
    while ((1 << s) < v) ++s;
    return (1 << s) == v ? s : -1;
}

// Checks that need no device data.  `for_accept` also checks vocab / path_stride.
int check_dims(const owl_dims* d, bool for_attn, bool for_accept) {
    if (!d) return OWL_ERR_INVALID_ARG;
    if (d->batch < 1 || d->total_nodes < d->batch || d->max_nodes < 1) return OWL_ERR_INVALID_ARG;
    if (d->max_nodes > kMaxNodes || d->batch > kMaxBatch) return OWL_ERR_UNSUPPORTED;
    if ((long long)d->max_nodes * d->batch < d->total_nodes) return OWL_ERR_INVALID_ARG;
    if (for_attn) {
        if (d->num_q_heads < 1 || d->num_kv_heads < 1 || d->num_q_heads % d->num_kv_heads != 0) return OWL_ERR_INVALID_ARG;
        if (d->num_kv_heads > 128) return OWL_ERR_UNSUPPORTED;
        if (d->max_pages_per_seq < 1 || d->num_pages < 1) return OWL_ERR_INVALID_ARG;
        if (!(d->sm_scale > 0.f) || d->sm_scale - d->sm_scale != 0.f) return OWL_ERR_INVALID_ARG;   // finite, > 0
        if (d->head_dim != kHeadDim) return OWL_ERR_UNSUPPORTED;
        if ((d->num_q_heads / d->num_kv_heads) * d->max_nodes > kMaxRows) return OWL_ERR_UNSUPPORTED;
        if (!(d->page_size == 16 || d->page_size == 32 || d->page_size == 64 || d->page_size == 128)) return OWL_ERR_UNSUPPORTED;
    }
    if (for_accept) {
        if (d->vocab < 1) return OWL_ERR_INVALID_ARG;
        if (d->path_stride < d->max_nodes) return OWL_ERR_INVALID_ARG;
    }
    return OWL_OK;
}

// One warp waits, with the kernels' own bounded wait, on an mbarrier that nothing ever completes.  The wait must
// give up after `limit_ns`, raise the abort flag (so that a second wait returns at once) and report kErrTimeout;
// the kernel then ends normally.  res[0]: nanoseconds the first wait took, res[1]: those of the second.
__global__ void selftest_wait_kernel(int32_t* status, unsigned long long limit_ns, unsigned long long* res) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        sm100::mbar_init(sm100::smem_u32(&bar), 1);
        abort_flag = 0;
        sm100::fence_barrier_init();
    }
    __syncthreads();
    const uint64_t t0 = sm100::global_timer_ns();
    const bool first = sm100::mbar_wait_ns(sm100::smem_u32(&bar), 0u, &abort_flag, limit_ns);
    const uint64_t t1 = sm100::global_timer_ns();
    const bool second = sm100::mbar_wait_ns(sm100::smem_u32(&bar), 0u, &abort_flag, limit_ns);
    const uint64_t t2 = sm100::global_timer_ns();
    if (threadIdx.x == 0) {
        if (!first && !second && abort_flag) report(status, kErrTimeout);
        res[0] = t1 - t0;
        res[1] = t2 - t1;
    }
}

// C[M, N] = A[M, K] B[N, K]^T on the tensor cores with one of the two epilogues (gemm_umma.cuh).
template <int kEpi>
static int launch_gemm(owl_ctx* ctx, const void* a, const void* b, int M, int N, int K, unsigned long long* row_key, float* c,
                       long long ldc, cudaStream_t stream) {
    gemm_path::GemmParams g{};
    g.M = M; g.N = N; g.K = K;
    g.row_blocks = (M + gemm_path::kBM - 1) / gemm_path::kBM;
    g.status = ctx->status;
    g.row_key = row_key; g.c = c; g.ldc = ldc;
    if (g.row_blocks == 2 && ctx->sm_count >= 2 && K % (2 * gemm_path::kBK) == 0) {
        // 129 to 256 rows: CTA pairs (gemm_umma_pair.cuh).  The columns are dealt out to the pairs as to single CTAs
        // below; a CTA stages half of a tile's rows of B.
        const int units = (N + 15) / 16, max_pairs = ctx->sm_count / 2;
        const int pairs = units < max_pairs ? units : max_pairs;
        const int per_pair = (units + pairs - 1) / pairs;
        g.rounds = (per_pair + 15) / 16;
        g.w_lo = per_pair / g.rounds * 16;
        g.wide_rounds = per_pair % g.rounds;
        g.a_bytes = gemm_path::kTileBytes;
        g.stage_bytes = 2 * (g.a_bytes + (g.w_lo + (g.wide_rounds ? 16 : 0)) / 2 * gemm_path::kBK * 2);   // two k-blocks
        const int fit = (gemm_path::kSmemLimit - gemm_path::kAuxBytes) / g.stage_bytes;
        g.stages = fit < gemm_path::kMaxStages ? fit : gemm_path::kMaxStages;
        CUtensorMap amap, bmap_hi, bmap_lo;
        const int ra = gemm_path::make_operand_map(ctx->encode, &amap, a, M, K, gemm_path::kBM);
        int rb = gemm_path::make_operand_map(ctx->encode, &bmap_lo, b, N, K, g.w_lo / 2);
        if (rb == 0) rb = g.wide_rounds ? gemm_path::make_operand_map(ctx->encode, &bmap_hi, b, N, K, (g.w_lo + 16) / 2) : (bmap_hi = bmap_lo, 0);
        if (ra != 0 || rb != 0) {
            snprintf(ctx->err, sizeof ctx->err, "cuTensorMapEncodeTiled failed (%d, %d): operands must be 16-byte aligned", ra, rb);
            return OWL_ERR_CUDA;
        }
        launch_dependent_smem(gemm_path::gemm_umma_pair_kernel<kEpi>, dim3(2u * (unsigned)pairs), dim3(gemm_path::kThreads),
                              (size_t)(gemm_path::kAuxBytes + g.stages * g.stage_bytes), stream, g, amap, bmap_hi, bmap_lo);
        ++ctx->launches;
        return OWL_OK;
    }
    // every CTA gets the same number of 16-column units, cut into as few tiles as the width limit allows
    const int units = (N + 15) / 16;
    const int grid = units < ctx->sm_count ? units : ctx->sm_count;
    const int per_cta = (units + grid - 1) / grid;
    const int wmax_units = gemm_path::max_tile_width(g.row_blocks) / 16;
    g.rounds = (per_cta + wmax_units - 1) / wmax_units;
    g.w_lo = per_cta / g.rounds * 16;
    g.wide_rounds = per_cta % g.rounds;
    // a stage: the rows of A that exist (the last row block rounded up to 8 rows) and the widest tile's rows of B
    const int last_rows = (M - (g.row_blocks - 1) * gemm_path::kBM + 7) / 8 * 8;
    g.a_bytes = (g.row_blocks - 1) * gemm_path::kTileBytes + last_rows * gemm_path::kBK * 2;
    g.stage_bytes = g.a_bytes + (g.w_lo + (g.wide_rounds ? 16 : 0)) * gemm_path::kBK * 2;
    g.stages = gemm_path::ring_stages(g.stage_bytes);
    CUtensorMap amap, amap_last, bmap_hi, bmap_lo;
    int ra = gemm_path::make_operand_map(ctx->encode, &amap, a, M, K, gemm_path::kBM);
    if (ra == 0) ra = gemm_path::make_operand_map(ctx->encode, &amap_last, a, M, K, last_rows);
    int rb = gemm_path::make_operand_map(ctx->encode, &bmap_lo, b, N, K, g.w_lo);
    if (rb == 0) rb = g.wide_rounds ? gemm_path::make_operand_map(ctx->encode, &bmap_hi, b, N, K, g.w_lo + 16) : (bmap_hi = bmap_lo, 0);
    if (ra != 0 || rb != 0) {
        snprintf(ctx->err, sizeof ctx->err, "cuTensorMapEncodeTiled failed (%d, %d): operands must be 16-byte aligned", ra, rb);
        return OWL_ERR_CUDA;
    }
    launch_dependent_smem(gemm_path::gemm_umma_kernel<kEpi>, dim3(grid), dim3(gemm_path::kThreads),
                          (size_t)gemm_path::smem_bytes(g.stages, g.stage_bytes), stream, g, amap, amap_last, bmap_hi, bmap_lo);
    ++ctx->launches;
    return OWL_OK;
}

}  // namespace

extern "C" {

const char* owl_status_string(int status) {
    switch (status) {
        case OWL_OK: return "ok";
        case OWL_ERR_INVALID_ARG: return "invalid argument";
        case OWL_ERR_UNSUPPORTED: return "unsupported shape";
        case OWL_ERR_CUDA: return "CUDA error";
        case OWL_ERR_BAD_TREE: return "malformed tree (device-detected)";
        case OWL_ERR_BAD_PAGE: return "page index or context length out of range (device-detected)";
        case OWL_ERR_TIMEOUT: return "bounded device wait expired";
        case OWL_ERR_TOO_LARGE: return "dims exceed the context's capacity";
        default: return "unknown status";
    }
}

const char* owl_last_error(const owl_ctx* ctx) { return ctx ? ctx->err : ""; }
int64_t owl_launch_count(const owl_ctx* ctx) { return ctx ? ctx->launches : 0; }

int owl_create(owl_ctx** out, int device, const owl_dims* max_dims) {
    if (!out || !max_dims) return OWL_ERR_INVALID_ARG;
    *out = nullptr;
    const bool attn = max_dims->num_q_heads > 0;
    const bool acc = max_dims->vocab > 0;
    int rc = check_dims(max_dims, attn, false);
    if (rc != OWL_OK) return rc;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return OWL_ERR_INVALID_ARG;

    owl_ctx* ctx = new (std::nothrow) owl_ctx();
    if (!ctx) return OWL_ERR_CUDA;
    ctx->device = device;
    ctx->max_dims = *max_dims;
    DeviceGuard guard(device);
    cudaError_t e;
    cudaDeviceProp prop;
    if ((e = cudaGetDeviceProperties(&prop, device)) != cudaSuccess) { delete ctx; return OWL_ERR_CUDA; }
    if (prop.major != 10) { delete ctx; return OWL_ERR_UNSUPPORTED; }  // sm_100a code only
    ctx->sm_count = prop.multiProcessorCount;
    ctx->num_ctas = ctx->sm_count;

    ctx->encode = load_encode_tiled();
    if (!ctx->encode) { delete ctx; return OWL_ERR_CUDA; }

    bool ok = true;
    auto alloc = [&](void** p, size_t bytes) {
        if (ok && (e = cudaMalloc(p, bytes ? bytes : 16)) != cudaSuccess) ok = false;
    };
    if (attn) {
        ctx->rows_per_slot = umma_path::kRows;
        ctx->slots = 2ll * ctx->num_ctas;      // a CTA stores at most two partials per call
        alloc((void**)&ctx->part_o, (size_t)ctx->slots * ctx->rows_per_slot * kHeadDim * sizeof(float));
        alloc((void**)&ctx->part_lse, (size_t)ctx->slots * ctx->rows_per_slot * sizeof(float));
    }
    alloc((void**)&ctx->status, sizeof(int32_t));
    alloc((void**)&ctx->selftest_ns, 2 * sizeof(unsigned long long));
    alloc((void**)&ctx->seq_bad, (size_t)max_dims->batch * sizeof(int32_t));
    alloc((void**)&ctx->sched_seq_begin, ((size_t)max_dims->batch + 1) * sizeof(long long));
    alloc((void**)&ctx->sched_header, sizeof(SchedHeader));
    if (acc) {
        ctx->part_keys_len = (long long)max_dims->total_nodes * ((max_dims->vocab + kArgmaxChunk - 1) / kArgmaxChunk);
        alloc((void**)&ctx->part_keys, (size_t)ctx->part_keys_len * sizeof(unsigned long long));
        alloc((void**)&ctx->lm_keys, 2 * (size_t)max_dims->total_nodes * sizeof(unsigned long long));
        if (ok) ok = cudaMemset(ctx->lm_keys, 0, 2 * (size_t)max_dims->total_nodes * sizeof(unsigned long long)) == cudaSuccess;
        alloc((void**)&ctx->seq_counter, 2 * (size_t)max_dims->batch * sizeof(unsigned int));
        if (ok) ok = cudaMemset(ctx->seq_counter, 0, 2 * (size_t)max_dims->batch * sizeof(unsigned int)) == cudaSuccess;
    }
    if (ok) {
        ok = cudaMemset(ctx->status, 0, sizeof(int32_t)) == cudaSuccess &&
             cudaMemset(ctx->seq_bad, 0, (size_t)max_dims->batch * sizeof(int32_t)) == cudaSuccess;
    }
    for (int i = 0; ok && i < 6; ++i) ok = cudaEventCreate(&ctx->ev[i]) == cudaSuccess;
    if (ok && attn) {
        ok = set_umma_smem_attr();
    }
    if (ok) {
        const int big = kCombineWarps * 32 * 32 * (int)sizeof(float4), small_ = big / 2;
        ok = cudaFuncSetAttribute(combine_sched_kernel<true, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize, big) == cudaSuccess &&
             cudaFuncSetAttribute(combine_sched_kernel<false, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize, big) == cudaSuccess &&
             cudaFuncSetAttribute(combine_sched_kernel<true, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, small_) == cudaSuccess &&
             cudaFuncSetAttribute(combine_sched_kernel<false, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, small_) == cudaSuccess;
    }
    if (ok) {
        ok = cudaFuncSetAttribute(gemm_path::gemm_umma_kernel<gemm_path::kEpiArgmax>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  gemm_path::kSmemLimit) == cudaSuccess &&
             cudaFuncSetAttribute(gemm_path::gemm_umma_kernel<gemm_path::kEpiStore>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  gemm_path::kSmemLimit) == cudaSuccess &&
             cudaFuncSetAttribute(gemm_path::gemm_umma_pair_kernel<gemm_path::kEpiArgmax>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  gemm_path::kSmemLimit) == cudaSuccess &&
             cudaFuncSetAttribute(gemm_path::gemm_umma_pair_kernel<gemm_path::kEpiStore>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  gemm_path::kSmemLimit) == cudaSuccess;
    }
    if (!ok || cudaDeviceSynchronize() != cudaSuccess) {
        cudaGetLastError();
        owl_destroy(ctx);
        return OWL_ERR_CUDA;
    }
    *out = ctx;
    return OWL_OK;
}

int owl_destroy(owl_ctx* ctx) {
    if (!ctx) return OWL_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaFree(ctx->part_o);
    cudaFree(ctx->part_lse);
    cudaFree(ctx->status);
    cudaFree(ctx->selftest_ns);
    cudaFree(ctx->seq_bad);
    cudaFree(ctx->sched_seq_begin);
    cudaFree(ctx->sched_header);
    cudaFree(ctx->part_keys);
    cudaFree(ctx->lm_keys);
    cudaFree(ctx->seq_counter);
    for (auto& s : ctx->stg) cudaFree(s.p);
    for (auto& ev : ctx->ev)
        if (ev) cudaEventDestroy(ev);
    delete ctx;
    return OWL_OK;
}

// Attention of a verify step.  `ap` non-null: the logits scan rides in the attention kernel's
// spare warps and the acceptance walk in the merge kernel, two launches for the whole step.
static int verify_attn_impl(owl_ctx* ctx, const owl_dims* d, const void* q, const void* k_cache, const void* v_cache,
                            const int32_t* block_table, const int32_t* ctx_lens, const int32_t* node_offsets,
                            const int32_t* tree_parent, void* out, float* lse, void* stream_, const AcceptParams* ap,
                            bool fp16 = false) {
    if (!ctx) return OWL_ERR_INVALID_ARG;
    int rc = check_dims(d, true, false);
    if (rc != OWL_OK) return rc;
    if (!q || !k_cache || !v_cache || !block_table || !ctx_lens || !tree_parent || !out) return OWL_ERR_INVALID_ARG;
    if (!node_offsets && d->total_nodes % d->batch != 0) return OWL_ERR_INVALID_ARG;
    if (!ctx->part_o) return OWL_ERR_TOO_LARGE;
    const owl_dims& mx = ctx->max_dims;
    const int G = d->num_q_heads / d->num_kv_heads;
    if (d->batch > mx.batch || d->total_nodes > mx.total_nodes) return OWL_ERR_TOO_LARGE;

    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    AttnParams p{};
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_cache = static_cast<const __nv_bfloat16*>(k_cache);
    p.v_cache = static_cast<const __nv_bfloat16*>(v_cache);
    p.block_table = block_table;
    p.ctx_lens = ctx_lens;
    p.node_offsets = node_offsets;
    p.tree_parent = tree_parent;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    p.part_o = ctx->part_o;
    p.part_lse = ctx->part_lse;
    p.status = ctx->status;
    p.seq_bad = ctx->seq_bad;
    p.sched_seq_begin = ctx->sched_seq_begin;
    p.sched_header = ctx->sched_header;
    p.epoch = ++ctx->epoch;
    p.batch = d->batch;
    p.total_nodes = d->total_nodes;
    p.nodes_uniform = d->total_nodes / d->batch;
    p.max_nodes = d->max_nodes;
    p.num_q_heads = d->num_q_heads;
    p.num_kv_heads = d->num_kv_heads;
    p.group = G;
    p.page_size = d->page_size;
    p.page_shift = log2_exact(d->page_size);
    p.max_pages_per_seq = d->max_pages_per_seq;
    p.num_pages = d->num_pages;
    p.rows_per_slot = ctx->rows_per_slot;
    p.num_ctas = ctx->num_ctas;
    p.sm_scale = d->sm_scale;
    p.f16 = fp16 ? 1 : 0;

    owl_ctx::MapEntry* maps = nullptr;
    {
        owl_ctx::MapEntry* lru = &ctx->maps[0];
        for (auto& m : ctx->maps) {
            if (m.k == k_cache && m.v == v_cache && m.pages == d->num_pages && m.heads == d->num_kv_heads &&
                m.page_size == d->page_size && m.fp16 == fp16) { maps = &m; break; }
            if (m.used < lru->used) lru = &m;
        }
        if (!maps) {
            const int rk = make_kv_tensor_map(ctx->encode, &lru->kmap, k_cache, d->num_pages, d->num_kv_heads, d->page_size, fp16);
            const int rv = make_kv_tensor_map(ctx->encode, &lru->vmap, v_cache, d->num_pages, d->num_kv_heads, d->page_size, fp16);
            if (rk != 0 || rv != 0) {
                lru->k = lru->v = nullptr;
                lru->used = 0;
                snprintf(ctx->err, sizeof ctx->err, "cuTensorMapEncodeTiled failed (%d, %d): caches must be 16-byte aligned", rk, rv);
                return OWL_ERR_CUDA;
            }
            lru->k = k_cache; lru->v = v_cache;
            lru->pages = d->num_pages; lru->heads = d->num_kv_heads; lru->page_size = d->page_size; lru->fp16 = fp16;
            maps = lru;
        }
        maps->used = ++ctx->map_clock;
    }

    if (ctx->profiling) cudaEventRecord(ctx->ev[0], stream);
    const long long rows = (long long)d->total_nodes * d->num_q_heads;
    // one warp per row up to two CTAs per SM; beyond that the merge kernel's warps stride over the rows
    const long long want_ctas = (rows + kCombineWarps - 1) / kCombineWarps;
    const unsigned grid = (unsigned)(want_ctas < 2ll * ctx->sm_count ? want_ctas : 2ll * ctx->sm_count);
    p.combine_row_ctas = (int32_t)grid;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(ctx->num_ctas);
        cfg.blockDim = dim3(umma_path::kThreads);
        cfg.dynamicSmemBytes = umma_path::kSmemBytes;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        // the instance that holds only this call's case: block-wide schedule above 32 sequences, the two-row-block
        // mode only if a unit (G * max_nodes rows at most) can exceed 128 rows, the logits scan only in a step
        const bool many = d->batch > 32, wide = G * d->max_nodes > 128;
        cudaLaunchKernelEx(&cfg, umma_kernel(many, wide, ap != nullptr, fp16), p, maps->kmap, maps->vmap, ap ? *ap : AcceptParams{});
    }
    ++ctx->launches;
    if (ctx->profiling) cudaEventRecord(ctx->ev[1], stream);
    const bool few_rows = rows <= 4096;      // latency-bound merge: 32 partials per round (see combine.cuh)
    const size_t stage_bytes = (size_t)kCombineWarps * (few_rows ? 32 : 16) * 32 * sizeof(float4);
    if (ap)
        launch_dependent_smem(few_rows ? combine_sched_kernel<true, 32> : combine_sched_kernel<true, 16>,
                              dim3(grid + (unsigned)d->batch), dim3(kCombineWarps * 32), stage_bytes, stream, p, *ap);
    else
        launch_dependent_smem(few_rows ? combine_sched_kernel<false, 32> : combine_sched_kernel<false, 16>, dim3(grid),
                              dim3(kCombineWarps * 32), stage_bytes, stream, p, AcceptParams{});
    ++ctx->launches;
    if (ctx->profiling) { cudaEventRecord(ctx->ev[2], stream); ctx->ev_attn_valid = true; }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_verify_attn launch");
    return OWL_OK;
}

int owl_verify_attn(owl_ctx* ctx, const owl_dims* d, const void* q, const void* k_cache, const void* v_cache,
                    const int32_t* block_table, const int32_t* ctx_lens, const int32_t* node_offsets,
                    const int32_t* tree_parent, void* out, float* lse, void* stream_) {
    return verify_attn_impl(ctx, d, q, k_cache, v_cache, block_table, ctx_lens, node_offsets, tree_parent, out, lse, stream_,
                            nullptr);
}

int owl_verify_attn_f16(owl_ctx* ctx, const owl_dims* d, const void* q, const void* k_cache, const void* v_cache,
                        const int32_t* block_table, const int32_t* ctx_lens, const int32_t* node_offsets,
                        const int32_t* tree_parent, void* out, float* lse, void* stream_) {
    return verify_attn_impl(ctx, d, q, k_cache, v_cache, block_table, ctx_lens, node_offsets, tree_parent, out, lse, stream_,
                            nullptr, true);
}

// Argument checks of the acceptance and its kernel parameters (everything but the counters of the stand-alone kernel).
static int accept_params(owl_ctx* ctx, const owl_dims* d, const float* logits, const int32_t* draft_tokens,
                         const int32_t* node_offsets, const int32_t* tree_parent, int32_t* accept_len,
                         int32_t* accept_path, int32_t* bonus_token, int32_t* node_argmax, AcceptParams& p,
                         int32_t* spec_node = nullptr) {
    if (!ctx) return OWL_ERR_INVALID_ARG;
    int rc = check_dims(d, false, true);
    if (rc != OWL_OK) return rc;
    if (!logits || !draft_tokens || !tree_parent || !accept_len || !accept_path || !bonus_token) return OWL_ERR_INVALID_ARG;
    if (!node_offsets && d->total_nodes % d->batch != 0) return OWL_ERR_INVALID_ARG;
    if (d->batch > ctx->max_dims.batch || d->total_nodes > ctx->max_dims.total_nodes) return OWL_ERR_TOO_LARGE;
    if (d->total_nodes > 65535) return OWL_ERR_UNSUPPORTED;
    const int chunks = (d->vocab + kArgmaxChunk - 1) / kArgmaxChunk;
    if (!ctx->part_keys || (long long)d->total_nodes * chunks > ctx->part_keys_len) return OWL_ERR_TOO_LARGE;
    p = AcceptParams{};
    p.logits = logits;
    p.draft_tokens = draft_tokens;
    p.node_offsets = node_offsets;
    p.tree_parent = tree_parent;
    p.accept_len = accept_len;
    p.accept_path = accept_path;
    p.bonus_token = bonus_token;
    p.node_argmax = node_argmax;
    p.spec_node = spec_node;
    p.part_keys = ctx->part_keys;
    p.chunks = chunks;
    p.status = ctx->status;
    p.batch = d->batch;
    p.total_nodes = d->total_nodes;
    p.nodes_uniform = d->total_nodes / d->batch;
    p.max_nodes = d->max_nodes;
    p.vocab = d->vocab;
    p.path_stride = d->path_stride;
    return OWL_OK;
}

static int tree_accept_impl(owl_ctx* ctx, const owl_dims* d, const float* logits, const int32_t* draft_tokens,
                            const int32_t* node_offsets, const int32_t* tree_parent, int32_t* accept_len,
                            int32_t* accept_path, int32_t* bonus_token, int32_t* spec_node, int32_t* node_argmax,
                            void* stream_) {
    AcceptParams p;
    const int rc = accept_params(ctx, d, logits, draft_tokens, node_offsets, tree_parent, accept_len, accept_path, bonus_token,
                                 node_argmax, p, spec_node);
    if (rc != OWL_OK) return rc;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int chunks = p.chunks;
    p.seq_counter = ctx->seq_counter;
    p.counter_stride = ctx->max_dims.batch;
    p.epoch = ++ctx->accept_epoch;
    if (ctx->profiling) cudaEventRecord(ctx->ev[3], stream);
    dim3 grid(argmax_grid((long long)chunks * d->total_nodes, ctx->sm_count));
    launch_dependent(argmax_partial_kernel, grid, dim3(kArgmaxThreads), stream, p);   // the walk runs in the CTA that finishes a sequence
    ++ctx->launches;
    if (ctx->profiling) cudaEventRecord(ctx->ev[4], stream);
    if (ctx->profiling) ctx->ev_accept_valid = true;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_tree_accept launch");
    return OWL_OK;
}

int owl_tree_accept(owl_ctx* ctx, const owl_dims* d, const float* logits, const int32_t* draft_tokens,
                    const int32_t* node_offsets, const int32_t* tree_parent, int32_t* accept_len,
                    int32_t* accept_path, int32_t* bonus_token, int32_t* node_argmax, void* stream_) {
    return tree_accept_impl(ctx, d, logits, draft_tokens, node_offsets, tree_parent, accept_len, accept_path, bonus_token,
                            nullptr, node_argmax, stream_);
}

int owl_tree_accept_spec(owl_ctx* ctx, const owl_dims* d, const float* logits, const int32_t* draft_tokens,
                         const int32_t* node_offsets, const int32_t* tree_parent, int32_t* accept_len,
                         int32_t* accept_path, int32_t* bonus_token, int32_t* spec_node, int32_t* node_argmax,
                         void* stream_) {
    if (!spec_node) return OWL_ERR_INVALID_ARG;
    return tree_accept_impl(ctx, d, logits, draft_tokens, node_offsets, tree_parent, accept_len, accept_path, bonus_token,
                            spec_node, node_argmax, stream_);
}

static int prepare_impl(owl_ctx* ctx, const owl_dims* d, const int32_t* node_offsets, const int32_t* tree_parent,
                        const int32_t* draft_tokens, const int32_t* ctx_lens, const int32_t* route, bool routed,
                        int32_t spec_token, int32_t* out_node_offsets, int32_t* out_tree_parent,
                        int32_t* out_draft_tokens, int32_t* out_input_ids, int32_t* out_position_ids, void* stream_) {
    if (!ctx) return OWL_ERR_INVALID_ARG;
    int rc = check_dims(d, false, false);
    if (rc != OWL_OK) return rc;
    // the prepared tree of a sequence with [SPEC] leaves has twice the nodes; a routed batch may also hold chains
    // of up to 64 nodes (kept as drafted), which the device sorts out per sequence
    if (!routed && 2 * d->max_nodes > kMaxNodes) return OWL_ERR_UNSUPPORTED;
    if (!tree_parent || !draft_tokens || !ctx_lens || !out_node_offsets || !out_tree_parent || !out_draft_tokens ||
        !out_input_ids || !out_position_ids || (routed && !route))
        return OWL_ERR_INVALID_ARG;
    if (!node_offsets && d->total_nodes % d->batch != 0) return OWL_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    PrepareParams p{};
    p.node_offsets = node_offsets; p.tree_parent = tree_parent; p.draft_tokens = draft_tokens; p.ctx_lens = ctx_lens;
    p.route = route;
    p.out_offsets = out_node_offsets; p.out_parent = out_tree_parent; p.out_draft = out_draft_tokens;
    p.out_input_ids = out_input_ids; p.out_position = out_position_ids;
    p.status = ctx->status;
    p.batch = d->batch; p.total_nodes = d->total_nodes; p.nodes_uniform = d->total_nodes / d->batch;
    p.max_nodes = d->max_nodes; p.spec_token = spec_token;
    launch_dependent(prepare_spec_kernel, dim3((unsigned)d->batch), dim3(kPrepareThreads), static_cast<cudaStream_t>(stream_), p);
    ++ctx->launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_prepare_spec_tree launch");
    return OWL_OK;
}

int owl_prepare_spec_tree(owl_ctx* ctx, const owl_dims* d, const int32_t* node_offsets, const int32_t* tree_parent,
                          const int32_t* draft_tokens, const int32_t* ctx_lens, int32_t spec_token,
                          int32_t* out_node_offsets, int32_t* out_tree_parent, int32_t* out_draft_tokens,
                          int32_t* out_input_ids, int32_t* out_position_ids, void* stream_) {
    return prepare_impl(ctx, d, node_offsets, tree_parent, draft_tokens, ctx_lens, nullptr, false, spec_token, out_node_offsets,
                        out_tree_parent, out_draft_tokens, out_input_ids, out_position_ids, stream_);
}

int owl_prepare_hybrid(owl_ctx* ctx, const owl_dims* d, const int32_t* node_offsets, const int32_t* tree_parent,
                       const int32_t* draft_tokens, const int32_t* ctx_lens, const int32_t* route, int32_t spec_token,
                       int32_t* out_node_offsets, int32_t* out_tree_parent, int32_t* out_draft_tokens,
                       int32_t* out_input_ids, int32_t* out_position_ids, void* stream_) {
    return prepare_impl(ctx, d, node_offsets, tree_parent, draft_tokens, ctx_lens, route, true, spec_token, out_node_offsets,
                        out_tree_parent, out_draft_tokens, out_input_ids, out_position_ids, stream_);
}

int owl_howl_route(int32_t batch, const float* score, float c, uint8_t* lastwaslinear, int32_t* route) {
    if (batch < 1 || !score || !lastwaslinear || !route || c != c) return OWL_ERR_INVALID_ARG;
    for (int32_t b = 0; b < batch; ++b) {
        const bool linear = score[b] > c;                      // a NaN score compares false: the tree drafter is used
        route[b] = linear ? OWL_ROUTE_LINEAR : (lastwaslinear[b] ? OWL_ROUTE_TREE_NOSPEC : OWL_ROUTE_TREE_SPEC);
        lastwaslinear[b] = linear ? 1 : 0;
    }
    return OWL_OK;
}

int owl_kv_commit(owl_ctx* ctx, const owl_dims* d, void* k_cache, void* v_cache, const int32_t* block_table,
                  int32_t* ctx_lens, const int32_t* node_offsets, const int32_t* accept_len, const int32_t* accept_path,
                  void* stream_) {
    if (!ctx) return OWL_ERR_INVALID_ARG;
    int rc = check_dims(d, false, false);
    if (rc != OWL_OK) return rc;
    if (d->num_kv_heads < 1 || d->max_pages_per_seq < 1 || d->num_pages < 1 || d->path_stride < 1) return OWL_ERR_INVALID_ARG;
    if (d->head_dim != kHeadDim || d->num_kv_heads > 128 ||
        !(d->page_size == 16 || d->page_size == 32 || d->page_size == 64 || d->page_size == 128))
        return OWL_ERR_UNSUPPORTED;
    if (!k_cache || !v_cache || !block_table || !ctx_lens || !accept_len || !accept_path) return OWL_ERR_INVALID_ARG;
    if (!node_offsets && d->total_nodes % d->batch != 0) return OWL_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    CommitParams p{};
    p.k_cache = static_cast<__nv_bfloat16*>(k_cache); p.v_cache = static_cast<__nv_bfloat16*>(v_cache);
    p.block_table = block_table; p.ctx_lens = ctx_lens; p.node_offsets = node_offsets;
    p.accept_len = accept_len; p.accept_path = accept_path; p.status = ctx->status;
    p.batch = d->batch; p.total_nodes = d->total_nodes; p.nodes_uniform = d->total_nodes / d->batch;
    p.max_nodes = d->max_nodes; p.num_kv_heads = d->num_kv_heads;
    p.page_size = d->page_size; p.page_shift = log2_exact(d->page_size);
    p.max_pages_per_seq = d->max_pages_per_seq; p.num_pages = d->num_pages; p.path_stride = d->path_stride;
    // the second kernel's wait is what keeps a length from being bumped while a CTA of the first still reads it
    launch_dependent(kv_commit_move_kernel, dim3(2u * (unsigned)d->num_kv_heads, (unsigned)d->batch), dim3(kCommitThreads), stream, p);
    launch_dependent(kv_commit_lens_kernel, dim3((unsigned)d->batch), dim3(kCommitThreads), stream, p);
    ctx->launches += 2;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_kv_commit launch");
    return OWL_OK;
}

int owl_lm_head_accept(owl_ctx* ctx, const owl_dims* d, int32_t hidden_dim, const void* hidden, const void* weight,
                       const int32_t* draft_tokens, const int32_t* node_offsets, const int32_t* tree_parent,
                       int32_t* accept_len, int32_t* accept_path, int32_t* bonus_token, int32_t* node_argmax, void* stream_) {
    if (!ctx) return OWL_ERR_INVALID_ARG;
    int rc = check_dims(d, false, true);
    if (rc != OWL_OK) return rc;
    if (!hidden || !weight || !draft_tokens || !tree_parent || !accept_len || !accept_path || !bonus_token) return OWL_ERR_INVALID_ARG;
    if (!node_offsets && d->total_nodes % d->batch != 0) return OWL_ERR_INVALID_ARG;
    if (hidden_dim < gemm_path::kBK) return OWL_ERR_INVALID_ARG;
    if (hidden_dim % gemm_path::kBK != 0 || d->total_nodes > gemm_path::kMaxRowBlocks * gemm_path::kBM) return OWL_ERR_UNSUPPORTED;
    if (!ctx->lm_keys || d->batch > ctx->max_dims.batch || d->total_nodes > ctx->max_dims.total_nodes) return OWL_ERR_TOO_LARGE;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    // The keys only ever grow (atomicMax) and must start from 0, below every real key.  Two sets alternate between
    // calls: this call's set was cleared, as a whole, by the walk kernel of the call before it (by owl_create for the
    // first two), and this call's walk kernel clears the other one - no memset in front of the product, which can
    // then queue up behind whatever kernel precedes it.  The call number moves on only once both kernels are launched.
    unsigned long long* keys = ctx->lm_keys + (size_t)(ctx->lm_epoch & 1u) * ctx->max_dims.total_nodes;
    unsigned long long* idle_keys = ctx->lm_keys + (size_t)((ctx->lm_epoch + 1u) & 1u) * ctx->max_dims.total_nodes;
    rc = launch_gemm<gemm_path::kEpiArgmax>(ctx, hidden, weight, d->total_nodes, d->vocab, hidden_dim, keys, nullptr, 0, stream);
    if (rc != OWL_OK) return rc;
    AcceptParams p{};
    p.draft_tokens = draft_tokens; p.node_offsets = node_offsets; p.tree_parent = tree_parent;
    p.accept_len = accept_len; p.accept_path = accept_path; p.bonus_token = bonus_token; p.node_argmax = node_argmax;
    p.part_keys = keys;
    p.chunks = 1;
    p.status = ctx->status;
    p.batch = d->batch; p.total_nodes = d->total_nodes; p.nodes_uniform = d->total_nodes / d->batch;
    p.max_nodes = d->max_nodes; p.vocab = d->vocab; p.path_stride = d->path_stride;
    launch_dependent(gemm_path::accept_walk_kernel, dim3((unsigned)d->batch), dim3(kArgmaxThreads), stream, p, idle_keys,
                     ctx->max_dims.total_nodes);
    ++ctx->launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_lm_head_accept launch");
    ++ctx->lm_epoch;
    return OWL_OK;
}

double owl_lstm_alpha(int32_t n_depth, int32_t d) {
    if (n_depth < 1 || d < 1) return 0.0;
    const double a0 = pow(2.0, -1.0 / (2.0 * n_depth));
    return 2.0 * a0 / ((1.0 - a0 * a0) * d);
}

int owl_lstm_cell(owl_ctx* ctx, int32_t rows, int32_t d_in, int32_t d, const void* h, const void* emb, const void* w, float alpha,
                  const float* ln_c_gamma, const float* ln_c_beta, const float* ln_z_gamma, const float* ln_z_beta, float eps,
                  float* z, float* h_out_f32, void* h_out_bf16, float* workspace, void* stream_) {
    if (!ctx || !h || !emb || !w || !z || !workspace || (!h_out_f32 && !h_out_bf16)) return OWL_ERR_INVALID_ARG;
    if (rows < 1 || d < 1 || d_in < gemm_path::kBK || !(eps >= 0.f) || alpha != alpha) return OWL_ERR_INVALID_ARG;
    if (d_in % gemm_path::kBK != 0 || rows > gemm_path::kMaxRowBlocks * gemm_path::kBM || d > kCellMaxD ||
        d % 4 != 0)
        return OWL_ERR_UNSUPPORTED;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int rc = launch_gemm<gemm_path::kEpiStore>(ctx, h, w, rows, 4 * d, d_in, nullptr, workspace, 4ll * d, stream);
    if (rc != OWL_OK) return rc;
    CellParams c{};
    c.s = workspace; c.emb = static_cast<const __nv_bfloat16*>(emb);
    c.gamma_c = ln_c_gamma; c.beta_c = ln_c_beta; c.gamma_z = ln_z_gamma; c.beta_z = ln_z_beta;
    c.z = z; c.h_f32 = h_out_f32; c.h_bf16 = static_cast<__nv_bfloat16*>(h_out_bf16);
    c.d = d; c.alpha = alpha; c.eps = eps;
    launch_dependent(lstm_cell_kernel, dim3((unsigned)rows * kCellCluster), dim3(kCellThreads), stream, c);
    ++ctx->launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_lstm_cell launch");
    return OWL_OK;
}

int owl_verify_step(owl_ctx* ctx, const owl_dims* d, const void* q, const void* k_cache, const void* v_cache,
                    const int32_t* block_table, const int32_t* ctx_lens, const int32_t* node_offsets,
                    const int32_t* tree_parent, void* out, float* lse, const float* logits, const int32_t* draft_tokens,
                    int32_t* accept_len, int32_t* accept_path, int32_t* bonus_token, int32_t* node_argmax, void* stream_) {
    if (!ctx) return OWL_ERR_INVALID_ARG;
    int rc = check_dims(d, true, true);
    if (rc != OWL_OK) return rc;
    // A scan of up to about a thousand (row, chunk) items - a few per spare warp - rides inside the attention kernel;
    // a larger one slows the attention down by more than its own kernel costs (measured: 4 x 64 nodes of a 128K
    // vocabulary, 570 -> 605 us), so it follows as a kernel of its own in stream order.
    const long long scan_items = (long long)d->total_nodes * ((d->vocab + kArgmaxChunk - 1) / kArgmaxChunk);
    if (scan_items > 1024) {
        rc = owl_verify_attn(ctx, d, q, k_cache, v_cache, block_table, ctx_lens, node_offsets, tree_parent, out, lse, stream_);
        if (rc != OWL_OK) return rc;
        return owl_tree_accept(ctx, d, logits, draft_tokens, node_offsets, tree_parent, accept_len, accept_path, bonus_token,
                               node_argmax, stream_);
    }
    // Two launches: the attention kernel, whose two spare warps per CTA scan the logits while K/V stream in, and the
    // merge kernel, which also walks the trees.
    AcceptParams ap;
    rc = accept_params(ctx, d, logits, draft_tokens, node_offsets, tree_parent, accept_len, accept_path, bonus_token, node_argmax, ap);
    if (rc != OWL_OK) return rc;
    ctx->ev_accept_valid = false;
    return verify_attn_impl(ctx, d, q, k_cache, v_cache, block_table, ctx_lens, node_offsets, tree_parent, out, lse, stream_, &ap);
}

int owl_verify_step_host(owl_ctx* ctx, const owl_dims* d, const void* q_h, const void* k_h, const void* v_h,
                         const int32_t* bt_h, const int32_t* cl_h, const int32_t* no_h, const int32_t* tp_h,
                         const float* logits_h, const int32_t* dt_h, void* out_h, float* lse_h, int32_t* alen_h,
                         int32_t* apath_h, int32_t* bonus_h, void* stream_) {
    if (!ctx) return OWL_ERR_INVALID_ARG;
    int rc = check_dims(d, true, true);
    if (rc != OWL_OK) return rc;
    if (!q_h || !k_h || !v_h || !bt_h || !cl_h || !tp_h || !logits_h || !dt_h || !out_h || !alen_h || !apath_h || !bonus_h)
        return OWL_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const size_t N = d->total_nodes, B = d->batch;
    const size_t q_bytes = N * d->num_q_heads * kHeadDim * 2;
    const size_t kv_bytes = (size_t)d->num_pages * d->num_kv_heads * d->page_size * kHeadDim * 2;
    const size_t sizes[16] = {q_bytes, kv_bytes, kv_bytes, B * d->max_pages_per_seq * 4, B * 4, (B + 1) * 4, N * 4,
                              N * (size_t)d->vocab * 4, N * 4,
                              /* outputs */ q_bytes, N * d->num_q_heads * 4, B * 4, B * (size_t)d->path_stride * 4, B * 4, 0, 0};
    for (int i = 0; i < 14; ++i) {
        if (ctx->stg[i].cap < sizes[i]) {
            cudaError_t e = cudaStreamSynchronize(stream);
            if (e == cudaSuccess) { cudaFree(ctx->stg[i].p); ctx->stg[i].p = nullptr; ctx->stg[i].cap = 0; e = cudaMalloc(&ctx->stg[i].p, sizes[i]); }
            if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_verify_step_host staging");
            ctx->stg[i].cap = sizes[i];
        }
    }
    const void* src[9] = {q_h, k_h, v_h, bt_h, cl_h, no_h, tp_h, logits_h, dt_h};
    for (int i = 0; i < 9; ++i) {
        if (!src[i]) continue;  // node_offsets may be NULL
        cudaError_t e = cudaMemcpyAsync(ctx->stg[i].p, src[i], sizes[i], cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_verify_step_host H2D");
    }
    auto dev = [&](int i) { return ctx->stg[i].p; };
    const int32_t* no_d = no_h ? static_cast<const int32_t*>(dev(5)) : nullptr;
    rc = owl_verify_step(ctx, d, dev(0), dev(1), dev(2), static_cast<const int32_t*>(dev(3)),
                         static_cast<const int32_t*>(dev(4)), no_d, static_cast<const int32_t*>(dev(6)), dev(9),
                         static_cast<float*>(dev(10)), static_cast<const float*>(dev(7)), static_cast<const int32_t*>(dev(8)),
                         static_cast<int32_t*>(dev(11)), static_cast<int32_t*>(dev(12)), static_cast<int32_t*>(dev(13)), nullptr,
                         stream_);
    if (rc != OWL_OK) return rc;
    void* dst[5] = {out_h, lse_h, alen_h, apath_h, bonus_h};
    for (int i = 0; i < 5; ++i) {
        if (!dst[i]) continue;
        cudaError_t e = cudaMemcpyAsync(dst[i], dev(9 + i), sizes[9 + i], cudaMemcpyDeviceToHost, stream);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_verify_step_host D2H");
    }
    return owl_get_status(ctx, stream_);
}

int owl_get_status(owl_ctx* ctx, void* stream_) {
    if (!ctx) return OWL_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int32_t st = 0;
    cudaError_t e = cudaMemcpyAsync(&st, ctx->status, sizeof st, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->status, 0, sizeof st, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_get_status");
    return st;
}

int owl_selftest_wait(owl_ctx* ctx, uint64_t limit_ns, uint64_t waited_ns[2], void* stream_) {
    if (!ctx || limit_ns == 0 || limit_ns > 1000000000ull) return OWL_ERR_INVALID_ARG;   // at most a second
    DeviceGuard guard(ctx->device);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    selftest_wait_kernel<<<1, 32, 0, stream>>>(ctx->status, limit_ns, ctx->selftest_ns);
    ++ctx->launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_selftest_wait launch");
    unsigned long long ns[2] = {0, 0};
    e = cudaMemcpyAsync(ns, ctx->selftest_ns, sizeof ns, cudaMemcpyDeviceToHost, stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_selftest_wait");
    const int st = owl_get_status(ctx, stream_);    // synchronises the stream
    if (waited_ns) { waited_ns[0] = ns[0]; waited_ns[1] = ns[1]; }
    return st;
}

int owl_set_profiling(owl_ctx* ctx, int on) {
    if (!ctx) return OWL_ERR_INVALID_ARG;
    ctx->profiling = on != 0;
    ctx->ev_attn_valid = ctx->ev_accept_valid = false;
    return OWL_OK;
}

int owl_last_kernel_times(owl_ctx* ctx, void* stream_, double t[4]) {
    if (!ctx || !t) return OWL_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream_));
    if (e != cudaSuccess) return cuda_fail(ctx, e, "owl_last_kernel_times");
    t[0] = t[1] = t[2] = t[3] = 0.0;
    float ms = 0.f;
    if (ctx->ev_attn_valid) {
        if (cudaEventElapsedTime(&ms, ctx->ev[0], ctx->ev[1]) == cudaSuccess) t[0] = ms * 1e-3;
        if (cudaEventElapsedTime(&ms, ctx->ev[1], ctx->ev[2]) == cudaSuccess) t[1] = ms * 1e-3;
    }
    if (ctx->ev_accept_valid) {
        if (cudaEventElapsedTime(&ms, ctx->ev[3], ctx->ev[4]) == cudaSuccess) t[2] = ms * 1e-3;
    }
    return OWL_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// owl_tree_accept_static: greedy tree acceptance for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they verify a draft: a
// serving engine that handed the whole device to its own pool allocator at start-up, a plug-in
// running inside someone else's memory budget, code on a latency path where an allocation (and
// the implicit device synchronisation it may bring) is not allowed.  owl_create allocates, so
// those callers cannot own an owl_ctx.  For them the arg-max scratch (one 64-bit key per logits
// row and 8192-float vocabulary chunk) and the device status word live in the fixed array below,
// which is part of the loaded library image: every device that loads the library holds its
// (OWL_STATIC_MAX_KEYS + 32 + 1024) * 8 bytes until the process exits, whether or not this entry point is ever called.
//
// The array's name is only a host-side handle here; the device address handed to the kernels
// comes from cudaGetSymbolAddress, looked up once per device with that device current.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxKeys = OWL_STATIC_MAX_KEYS;            // (row, chunk) keys
constexpr int kStaticStatusWords = 32;                         // one 256-byte line for the status word
constexpr int kStaticCounterWords = kMaxBatch;                 // per-sequence progress counters of the scan
constexpr int kStaticMaxDevices = 64;

static __device__ __align__(256) unsigned long long g_accept_scratch[kStaticMaxKeys + kStaticStatusWords + kStaticCounterWords];
// Every device has its own copy of the array, hence its own call counter: the counter's parity selects the set of
// progress counters a call counts in, and the set a call clears must be the one the next call ON THAT DEVICE uses.
unsigned long long* g_static_addr[kStaticMaxDevices] = {nullptr};
bool g_static_ready[kStaticMaxDevices] = {false};
uint32_t g_static_epoch[kStaticMaxDevices] = {0};
std::mutex g_static_mutex;

// Device address of g_accept_scratch on the current device `dev` (looked up on first use) and the number of this
// call among the calls made on that device.
cudaError_t static_scratch(int dev, unsigned long long** out, uint32_t* epoch) {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ready[dev]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_accept_scratch);
        if (e != cudaSuccess) return e;
        g_static_addr[dev] = static_cast<unsigned long long*>(p);
        g_static_ready[dev] = true;
    }
    *out = g_static_addr[dev];
    *epoch = ++g_static_epoch[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int owl_tree_accept_static(const owl_dims* d, const float* logits, const int32_t* draft_tokens,
                                      const int32_t* node_offsets, const int32_t* tree_parent, int32_t* accept_len,
                                      int32_t* accept_path, int32_t* bonus_token, int32_t* node_argmax,
                                      int32_t* device_status, void* stream_) {
    int rc = check_dims(d, false, true);
    if (rc != OWL_OK) return rc;
    if (!logits || !draft_tokens || !tree_parent || !accept_len || !accept_path || !bonus_token) return OWL_ERR_INVALID_ARG;
    if (!node_offsets && d->total_nodes % d->batch != 0) return OWL_ERR_INVALID_ARG;
    if (d->total_nodes > 65535) return OWL_ERR_UNSUPPORTED;
    const int chunks = (d->vocab + kArgmaxChunk - 1) / kArgmaxChunk;
    if ((long long)d->total_nodes * chunks > kStaticMaxKeys) return OWL_ERR_TOO_LARGE;   // beyond the fixed scratch

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return OWL_ERR_CUDA;
    unsigned long long* scratch = nullptr;
    uint32_t epoch = 0;
    if (static_scratch(dev, &scratch, &epoch) != cudaSuccess) { cudaGetLastError(); return OWL_ERR_CUDA; }
    // without a status word of the caller's the verdict goes to a word of the array that no call reports
    int32_t* status = device_status ? device_status : reinterpret_cast<int32_t*>(scratch + kStaticMaxKeys);

    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    // The keys need no clearing (every key a call reads it has written first); the status word does.
    if (cudaMemsetAsync(status, 0, sizeof(int32_t), stream) != cudaSuccess) { cudaGetLastError(); return OWL_ERR_CUDA; }
    AcceptParams p{};
    p.logits = logits;
    p.draft_tokens = draft_tokens;
    p.node_offsets = node_offsets;
    p.tree_parent = tree_parent;
    p.accept_len = accept_len;
    p.accept_path = accept_path;
    p.bonus_token = bonus_token;
    p.node_argmax = node_argmax;
    p.part_keys = scratch;
    p.chunks = chunks;
    p.status = status;
    p.batch = d->batch;
    p.total_nodes = d->total_nodes;
    p.nodes_uniform = d->total_nodes / d->batch;
    p.max_nodes = d->max_nodes;
    p.vocab = d->vocab;
    p.path_stride = d->path_stride;
    p.seq_counter = reinterpret_cast<unsigned int*>(scratch + kStaticMaxKeys + kStaticStatusWords);   // 2 x kMaxBatch
    p.counter_stride = kMaxBatch;
    p.epoch = epoch;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) { cudaGetLastError(); return OWL_ERR_CUDA; }
    argmax_partial_kernel<<<argmax_grid((long long)chunks * d->total_nodes, sms), kArgmaxThreads, 0, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return OWL_ERR_CUDA;
    return OWL_OK;
}
