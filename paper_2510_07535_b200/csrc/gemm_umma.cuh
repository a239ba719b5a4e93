// Weight-streaming product C[M, N] = A[M, K] B[N, K]^T on the 5th-generation tensor cores (bf16 operands,
// fp32 accumulators in tensor memory), for the two producers either side of the verify step:
//   LM head     A = hidden states of the drafted nodes [nodes, 4096], B = head weight [vocab, 4096]; the epilogue
//               keeps of every row only its arg-max over the vocabulary - the logits are never written;
//   drafter     A = h [rows, d_in], B = [W^f; W^i; W^o; W^c] ([4d, d_in]), Eq. 2; the epilogue stores fp32.
// M is small (up to 384 rows: 1 to 3 blocks of 128), N is huge: B is read from HBM exactly once, A comes again and
// again out of L2.  One persistent CTA per SM takes column tiles of C round-robin:
//   warp 0     TMA producer: per 64-wide k-block one box per row block of A and one or two boxes of B into a ring
//   warp 1     issues the tcgen05.mma (one thread): per k-block 4 k-steps x row blocks, 128 x width x 16 each
//   warps 4-7  epilogue, thread = row: reads its accumulators of every row block and reduces or stores them
// Tile width.  A 128 x 128 x 16 instruction reads 4 KB of A and 4 KB of B from shared memory in its 64 clocks, which
// together with the TMA writes is more than the 128 B / clock shared memory delivers: two row blocks ran at 875
// clocks per k-block for 512 of tensor-pipe time.  A 128 x 256 x 16 instruction reads 12 KB in 128 clocks, so up to
// two row blocks take tiles of up to 256 columns (all 512 columns of tensor memory as one accumulator buffer for two
// row blocks, two buffers for one); three row blocks take up to 160 (3 x 160 = 480 columns: 7-9 % faster than 128).
// Balance.  B is read once and every CTA streams at the same rate, so the columns are dealt out evenly: each CTA
// gets ceil(N / 16 / CTAs) units of 16 columns, cut into as few tiles as the width limit allows, the tiles of one
// round equally wide on every CTA (widths differ by at most 16 between rounds).  The instruction's N is the tile
// width (any multiple of 16), one TMA box brings the tile's rows of B.  N = 49152 on 148 CTAs: rounds of 176 and
// 160 columns, 98.8 % of the last round filled, against 65 % with 256-wide tiles only.
// Ring.  At 6.5 TB/s over 148 SMs and 2.5-3 us of loaded memory latency a CTA needs 110-130 KB of B in flight, so a
// stage holds what is loaded and nothing else: the tile's rows of B and the valid rows of A rounded up to 8 (one
// swizzle atom).  The instruction still reads 128 rows of A: past the loaded ones it finds whatever follows in
// shared memory (the stage's B, the next stage, the pad behind the ring), which only feeds accumulator rows >= M that
// nobody reads - an output row depends on its own row of A alone.  10 rows against 176 of B: 24 KB per stage, 8
// stages, 176 KB in flight (with 48 KB stages there were 88 KB in flight and the product ran at 4.2 TB/s).
// Every wait is bounded as in the attention kernel.
#pragma once

#include <cuda.h>
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "accept.cuh"
#include "kv_tensor_map.cuh"
#include "owl_common.cuh"
#include "sm100_ptx.cuh"

namespace owl {
namespace gemm_path {

using namespace sm100;

constexpr int kBM = 128, kBN = 128, kBK = 64;
constexpr int kThreads = 256;
constexpr int kTileBytes = kBM * kBK * 2;        // 16 KB: 128 rows of one 128-byte swizzle row each
constexpr int kMaxRowBlocks = 3;
constexpr int kMaxStages = 12;
constexpr int kAuxBytes = 1024;
constexpr int kSmemLimit = 232448;               // 227 KB

enum Epilogue { kEpiArgmax = 0, kEpiStore = 1 };

struct GemmParams {
    int M, N, K;
    int row_blocks;                 // ceil(M / 128)
    int stages;                     // ring depth: what fits beside the aux area and the pad
    int a_bytes;                    // per stage: full row blocks of 16 KB, then the last block's rows rounded up to 8
    int stage_bytes;                // a_bytes + the widest tile's rows of B, 128 bytes each
    int rounds;                     // tiles per CTA; round t holds one tile per CTA, all of the same width
    int wide_rounds;                // rounds [0, wide_rounds) are w_lo + 16 columns wide, the others w_lo
    int w_lo;                       // multiple of 16, <= 256 (160 with three row blocks)
    int32_t* status;
    unsigned long long* row_key;    // kEpiArgmax: [M] keys (value, ~column), raised by atomicMax; cleared by the caller
    float* c;                       // kEpiStore: fp32 [M, ldc]
    long long ldc;
};

struct Aux {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Aux) <= kAuxBytes, "aux area too small");

// up to two row blocks take tiles of 256 columns, three of 128 (tensor memory: row blocks x width <= 512 columns)
// widest tile: row blocks x width columns of fp32 accumulators must fit the 512 columns of tensor memory
__host__ __device__ inline int max_tile_width(int row_blocks) { return row_blocks <= 2 ? 256 : 160; }
// shared memory: [aux][stages x stage_bytes][pad: the A operand window of the last stage may reach one tile past it]
__host__ inline int ring_stages(int stage_bytes) {
    const int s = (kSmemLimit - kAuxBytes - kTileBytes) / stage_bytes;
    return s < kMaxStages ? s : kMaxStages;
}
__host__ inline int smem_bytes(int stages, int stage_bytes) { return kAuxBytes + stages * stage_bytes + kTileBytes; }

// 2-D tile load global -> shared with an L2 cache policy, completion counted in bytes on an mbarrier of this CTA.
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        : : "r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

template <int kEpi>
__global__ void __launch_bounds__(kThreads, 1)
gemm_umma_kernel(const GemmParams p, const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap amap_last,
                 const __grid_constant__ CUtensorMap bmap_hi, const __grid_constant__ CUtensorMap bmap_lo) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = smem_u32(smem) + kAuxBytes;       // the ring
    const int rb = p.row_blocks, stages = p.stages;
    const int sbytes = p.stage_bytes;
    Aux* aux = reinterpret_cast<Aux*>(smem);
    volatile int* abort_flag = &aux->abort_flag;
    if (smem_base & 1023u) {                       // operand tiles must sit on swizzle-atom boundaries
        if (tid == 0) report(p.status, kErrTimeout);
        return;
    }
    if (tid == 0) {
        for (int i = 0; i < stages; ++i) { mbar_init(smem_u32(&aux->full[i]), 1); mbar_init(smem_u32(&aux->empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&aux->acc_full[i]), 1); mbar_init(smem_u32(&aux->acc_empty[i]), 128); }
        aux->abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&amap);
        tma_prefetch_desc(&amap_last);
        tma_prefetch_desc(&bmap_hi);
        tma_prefetch_desc(&bmap_lo);
    }
    if (warp == 0) { tmem_alloc(smem_u32(&aux->tmem_base), 512); tmem_relinquish(); }
    // may be launched as a programmatic dependent of the kernel before it in the stream: the set-up above touched no
    // input and ran beside that kernel's tail; from here on it has completed (a no-op in an ordinary launch).  The
    // kernel after this one may queue up in turn; it waits likewise before it reads anything.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = aux->tmem_base;
    const int kblocks = p.K / kBK;
    const int wmax = max_tile_width(rb);         // widest tile: 256 columns, 160 with three row blocks
    const int nbuf = rb * wmax * 2 <= 512 ? 2 : 1; // accumulator buffers of rb x wmax columns each
    // round t: one tile per CTA, the rounds' column bands one after the other; a tile that starts past N is empty
    auto tile_width = [&](int t) { return t < p.wide_rounds ? p.w_lo + 16 : p.w_lo; };
    auto tile_col0 = [&](int t) {
        const int hi = t < p.wide_rounds ? t : p.wide_rounds;
        return (int)gridDim.x * (hi * (p.w_lo + 16) + (t - hi) * p.w_lo) + (int)blockIdx.x * tile_width(t);
    };
    uint32_t issued = 0;

    if (warp == 0) {
        if (lane == 0) {
            const uint64_t stream_policy = l2_policy_evict_first();   // B is read once
            const uint64_t keep_policy = l2_policy_evict_last();      // A is read by every CTA for every tile
            uint32_t it = 0;
            for (int t = 0; t < p.rounds; ++t) {
                const int col0 = tile_col0(t), w = tile_width(t);
                if (col0 >= p.N) break;
                const CUtensorMap* bmap = t < p.wide_rounds ? &bmap_hi : &bmap_lo;   // box = the tile's w rows of B
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t stage = it % stages, ph = (it / stages) & 1u;
                    if (!mbar_wait(smem_u32(&aux->empty[stage]), ph ^ 1u, abort_flag)) continue;
                    const uint32_t full = smem_u32(&aux->full[stage]);
                    const uint32_t dst = smem_base + stage * sbytes;
                    mbar_arrive_expect_tx(full, (uint32_t)(p.a_bytes + w * kBK * 2));
                    for (int r = 0; r < rb; ++r)       // the last row block's box is as high as its valid rows (rounded up to 8)
                        tma_load_2d_hint(dst + r * kTileBytes, r + 1 < rb ? &amap : &amap_last, full, kb * kBK, r * kBM, keep_policy);
                    tma_load_2d_hint(dst + p.a_bytes, bmap, full, kb * kBK, col0, stream_policy);
                    issued = it + 1;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t it = 0, tcount = 0;
            for (int t = 0; t < p.rounds; ++t, ++tcount) {
                if (tile_col0(t) >= p.N) break;
                const uint32_t buf = tcount % nbuf, acc_ph = (tcount / nbuf) & 1u;
                const uint32_t idesc = umma_idesc_16bit(kBM, tile_width(t), 0, 0, false);
                bool ok = mbar_wait(smem_u32(&aux->acc_empty[buf]), acc_ph ^ 1u, abort_flag);   // the epilogue has read this buffer
                tc_fence_after();
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t stage = it % stages, ph = (it / stages) & 1u;
                    ok = mbar_wait(smem_u32(&aux->full[stage]), ph, abort_flag) && ok;
                    tc_fence_after();
                    if (ok) {
                        const uint32_t a0 = smem_base + stage * sbytes;
                        const uint64_t bdesc = umma_smem_desc_sw128(a0 + p.a_bytes, 16, 1024);
                        for (int r = 0; r < rb; ++r) {
                            const uint64_t adesc = umma_smem_desc_sw128(a0 + r * kTileBytes, 16, 1024);
                            const uint32_t d = tmem + buf * (uint32_t)(rb * wmax) + r * wmax;
#pragma unroll
                            for (int ks = 0; ks < kBK / 16; ++ks)    // 32 bytes along K inside the 128-byte swizzle row
                                umma_ss(d, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), idesc, (kb | ks) ? 1u : 0u);
                        }
                        umma_commit(smem_u32(&aux->empty[stage]));
                    }
                }
                if (ok) umma_commit(smem_u32(&aux->acc_full[buf]));
            }
        }
    } else if (warp >= 4) {
        const int lane_row = (warp & 3) * 32 + lane;                    // TMEM lane = row inside a row block
        const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
        uint32_t tcount = 0;
        for (int t = 0; t < p.rounds; ++t, ++tcount) {
            const int n0 = tile_col0(t);
            if (n0 >= p.N) break;
            const uint32_t buf = tcount % nbuf, acc_ph = (tcount / nbuf) & 1u;
            const bool ok = mbar_wait(smem_u32(&aux->acc_full[buf]), acc_ph, abort_flag);
            tc_fence_after();
            // columns [n0, n_end) are this tile's; a width that is an odd multiple of 16 leaves half of the last chunk
            // of 32 unused (those columns of tensor memory hold another tile's or no data)
            const int n_end = n0 + tile_width(t) < p.N ? n0 + tile_width(t) : p.N;
            const int chunks = (tile_width(t) + 31) / 32;
            for (int r = 0; r < rb; ++r) {
                const int row = r * kBM + lane_row;
                const uint32_t taddr = tmem + lane_sel + buf * (uint32_t)(rb * wmax) + r * wmax;
                float bv = -INFINITY;
                uint32_t bi = 0xffffffffu;
#pragma unroll 1
                for (int c4 = 0; c4 < chunks; ++c4) {
                    uint32_t v[32];
                    tmem_ld32(taddr + c4 * 32, v);
                    tmem_wait_ld();
                    if (!ok || row >= p.M) continue;
                    const int col0 = n0 + c4 * 32;
                    if (kEpi == kEpiArgmax) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            // NaN reads as -inf; strict '>' keeps the lowest column among equal values
                            const float x = __uint_as_float(v[j]);
                            const float e = x != x ? -INFINITY : x;
                            if (col0 + j < n_end && (bi == 0xffffffffu || e > bv)) { bv = e; bi = (uint32_t)(col0 + j); }
                        }
                    } else {
                        float* dst = p.c + (long long)row * p.ldc + col0;
                        if (col0 + 32 <= n_end && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                reinterpret_cast<uint4*>(dst)[j] = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                        } else {
                            for (int j = 0; j < 32 && col0 + j < n_end; ++j) dst[j] = __uint_as_float(v[j]);
                        }
                    }
                }
                if (kEpi == kEpiArgmax && ok && row < p.M && bi != 0xffffffffu) atomicMax(p.row_key + row, argmax_key(bv, bi));
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&aux->acc_empty[buf]));    // unconditional: the issuing thread's wait must end
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        if (aux->abort_flag) {
            // give the copies still in flight a bounded time to land before the CTA's shared memory is released
            if (lane == 0) {
                const uint32_t first = issued > (uint32_t)stages ? issued - stages : 0u;
                for (uint32_t it = first; it < issued; ++it) {
                    const uint32_t bar = smem_u32(&aux->full[it % stages]), ph = (it / stages) & 1u;
                    for (int polls = 0; polls < (1 << 20) && !mbar_try_wait(bar, ph); ++polls) {}
                }
                report(p.status, kErrTimeout);
            }
            __syncwarp();
        }
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}

// Row-major bf16 matrix [rows, K] as a 2-D tensor map with boxes of 64 columns x box_rows rows (128-byte swizzle; a
// multiple of 8 rows up to 256): one box is one operand tile in the canonical K-major layout.  Rows past the end read
// as zeros.
inline int make_operand_map(EncodeTiledFn encode, CUtensorMap* map, const void* ptr, long long rows, long long K, int box_rows) {
    if (!encode) return -1;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {kBK, (cuuint32_t)box_rows};
    const cuuint32_t elem_strides[2] = {1, 1};
    return (int)encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, elem_strides,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// One sequence's acceptance walk per CTA over one key per row (the arg-max the product's epilogue left).  The grid
// also clears `idle_keys[0, idle_len)`, the key set the next call's product will raise (nothing of this call uses it).
// Launched as a programmatic dependent of the product: it reads nothing before the product has completed.
__global__ void __launch_bounds__(kArgmaxThreads) accept_walk_kernel(const AcceptParams p, unsigned long long* idle_keys, int idle_len) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int i = blockIdx.x * kArgmaxThreads + threadIdx.x; i < idle_len; i += gridDim.x * kArgmaxThreads) idle_keys[i] = 0ull;
    accept_walk_seq(p, (int)blockIdx.x);
}

}  // namespace gemm_path

// ------------------------------------------------------------------------------------------------------------
// The drafter cell's element-wise half (Eq. 2, 5-8) over the fp32 pre-activations
// S = h [W^f; W^i; W^o; W^c]^T ([rows, 4d]).  f = layer normalisation (biased variance, eps inside the root,
// optional affine) followed by exact GeLU.
// A row is spread over a cluster of 8 CTAs (a handful of rows would otherwise sit on a handful of SMs: 10 rows of
// 12288 took 30 us on one CTA each).  The statistics of the two layer normalisations are over the whole row: one
// exchange through distributed shared memory and one cluster barrier each (cluster_mean_rstd).
// ------------------------------------------------------------------------------------------------------------
constexpr int kCellCluster = 8;
constexpr int kCellThreads = 512;
constexpr int kCellPerThread = 4;                // d <= 8 * 512 * 4 = 16384
constexpr int kCellMaxD = kCellCluster * kCellThreads * kCellPerThread;

struct CellParams {
    const float* s;                  // [rows, 4d]: W^f h, W^i h, W^o h, W^c h
    const __nv_bfloat16* emb;        // [rows, d]  E(t), Eq. 1
    const float* gamma_c; const float* beta_c;   // affine of f in Eq. 6 (may be null)
    const float* gamma_z; const float* beta_z;   // affine of f in Eq. 8 (may be null)
    float* z;                        // [rows, d] in / out
    float* h_f32;                    // [rows, d] out (may be null)
    __nv_bfloat16* h_bf16;           // [rows, d] out (may be null)
    int d;
    float alpha, eps;
};

// Sum of v over the CTA's threads; s_warp is free again after the second barrier.
__device__ __forceinline__ float cell_block_sum(float v, float* s_warp) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) s_warp[warp] = v;
    __syncthreads();
    float t = lane < kCellThreads / 32 ? s_warp[lane] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    __syncthreads();
    return t;
}

// Mean and 1 / sqrt(variance + eps) over a whole row from the values x[] this thread holds (on[] says which exist).
// Each CTA takes the mean and the sum of squared deviations of its own `count` columns (two block reductions), pushes
// the pair into slot `which` of every CTA of the cluster, and after one cluster barrier all of them combine the eight
// pairs in rank order by the pairwise-variance identity  M2 = sum_i M2_i + sum_i n_i (mean_i - mean)^2 : the same
// numbers everywhere, no cancellation, and nobody reads a peer's shared memory after the barrier.
__device__ __forceinline__ void cluster_mean_rstd(const float (&x)[kCellPerThread], const bool (&on)[kCellPerThread], int count,
                                                  int slice, int d, float eps, float* s_warp, float (*s_stat)[kCellCluster][2],
                                                  int which, float& mean, float& rstd) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    float sum = 0.f;
#pragma unroll
    for (int k = 0; k < kCellPerThread; ++k) sum += on[k] ? x[k] : 0.f;
    const float mean_cta = count > 0 ? cell_block_sum(sum, s_warp) / count : (cell_block_sum(sum, s_warp), 0.f);
    float sq = 0.f;
#pragma unroll
    for (int k = 0; k < kCellPerThread; ++k)
        if (on[k]) { const float t = x[k] - mean_cta; sq += t * t; }
    const float m2_cta = cell_block_sum(sq, s_warp);
    const int rank = (int)cluster.block_rank();
    if (threadIdx.x < kCellCluster) {
        float* dst = &cluster.map_shared_rank(s_stat, threadIdx.x)[which][rank][0];
        dst[0] = mean_cta;
        dst[1] = m2_cta;
    }
    cluster.sync();
    float total = 0.f;
#pragma unroll
    for (int r = 0; r < kCellCluster; ++r) {
        const int n_r = min(slice, max(d - r * slice, 0));
        total += (float)n_r * s_stat[which][r][0];
    }
    mean = total / d;
    float m2 = 0.f;
#pragma unroll
    for (int r = 0; r < kCellCluster; ++r) {
        const int n_r = min(slice, max(d - r * slice, 0));
        const float dm = s_stat[which][r][0] - mean;
        m2 += s_stat[which][r][1] + (float)n_r * dm * dm;
    }
    rstd = rsqrtf(m2 / d + eps);
}

__device__ __forceinline__ float gelu_exact(float x) { return 0.5f * x * (1.f + erff(x * 0.70710678118654752f)); }
__device__ __forceinline__ float sigmoid_f(float x) { return 1.f / (1.f + __expf(-x)); }

__global__ void __cluster_dims__(kCellCluster, 1, 1) __launch_bounds__(kCellThreads) lstm_cell_kernel(const CellParams p) {
    namespace cg = cooperative_groups;
    __shared__ float s_warp[kCellThreads / 32];
    __shared__ float s_stat[2][kCellCluster][2];     // [which normalisation][CTA of the cluster][mean, M2]
    cg::cluster_group cluster = cg::this_cluster();
    // may be launched as a programmatic dependent of the product that writes S; the kernel after this one may queue up
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long row = blockIdx.x / kCellCluster;
    const int d = p.d;
    const int slice = (d + kCellCluster - 1) / kCellCluster;
    const int j0 = (int)cluster.block_rank() * slice;             // this CTA's columns: [j0, min(j0 + slice, d))
    const int count = min(slice, max(d - j0, 0));
    const float* s = p.s + row * 4ll * d;
    // everything a column needs is asked for at once: the four pre-activations, E(t) and z
    float xc[kCellPerThread], sf[kCellPerThread], si[kCellPerThread], so[kCellPerThread], zo[kCellPerThread], zn[kCellPerThread];
    bool on[kCellPerThread];
#pragma unroll
    for (int k = 0; k < kCellPerThread; ++k) {
        const int i = k * kCellThreads + threadIdx.x, j = j0 + i;
        on[k] = i < slice && j < d;
        xc[k] = sf[k] = si[k] = so[k] = zo[k] = zn[k] = 0.f;
        if (on[k]) {
            const float ae = p.alpha * __bfloat162float(p.emb[row * d + j]);     // s^m = W^m h + alpha e  (Eq. 2)
            sf[k] = s[j] + ae; si[k] = s[1ll * d + j] + ae; so[k] = s[2ll * d + j] + ae; xc[k] = s[3ll * d + j] + ae;
            zo[k] = p.z[row * d + j];
        }
    }
    cluster.sync();      // every CTA of the cluster is running before anyone writes into its shared memory (the loads fly)
    float mean_c, rstd_c;
    cluster_mean_rstd(xc, on, count, slice, d, p.eps, s_warp, s_stat, 0, mean_c, rstd_c);
    // z' = z g^f + f(s^c) g^i  (Eq. 5-7)
#pragma unroll
    for (int k = 0; k < kCellPerThread; ++k) {
        const int j = j0 + k * kCellThreads + threadIdx.x;
        if (on[k]) {
            float y = (xc[k] - mean_c) * rstd_c;
            if (p.gamma_c) y *= p.gamma_c[j];
            if (p.beta_c) y += p.beta_c[j];
            zn[k] = zo[k] * sigmoid_f(sf[k]) + gelu_exact(y) * sigmoid_f(si[k]);
            p.z[row * d + j] = zn[k];
        }
    }
    float mean_z, rstd_z;
    cluster_mean_rstd(zn, on, count, slice, d, p.eps, s_warp, s_stat, 1, mean_z, rstd_z);
    // h' = f(z') g^o  (Eq. 8)
#pragma unroll
    for (int k = 0; k < kCellPerThread; ++k) {
        const int j = j0 + k * kCellThreads + threadIdx.x;
        if (on[k]) {
            float y = (zn[k] - mean_z) * rstd_z;
            if (p.gamma_z) y *= p.gamma_z[j];
            if (p.beta_z) y += p.beta_z[j];
            const float h = gelu_exact(y) * sigmoid_f(so[k]);
            if (p.h_f32) p.h_f32[row * d + j] = h;
            if (p.h_bf16) p.h_bf16[row * d + j] = __float2bfloat16_rn(h);
        }
    }
}

}  // namespace owl
