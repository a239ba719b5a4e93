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
// two row blocks take 256-column tiles (all 512 columns of tensor memory as one accumulator buffer for two row
// blocks, two buffers for one) - as many full rounds of them as the grid has CTAs, the rest of the columns in
// 128-wide tiles, so that the last round is not a quarter empty.  Three row blocks take 128-wide tiles throughout.
// Every wait is bounded as in the attention kernel.
#pragma once

#include <cuda.h>
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
constexpr int kMaxStages = 8;
constexpr int kAuxBytes = 1024;
constexpr int kSmemLimit = 232448;               // 227 KB

enum Epilogue { kEpiArgmax = 0, kEpiStore = 1 };

struct GemmParams {
    int M, N, K;
    int row_blocks;                 // ceil(M / 128)
    int stages;                     // ring depth: what fits beside the aux area
    int wide_tiles;                 // tiles [0, wide_tiles) are 256 columns wide, the others 128
    int n_tiles;                    // wide_tiles + ceil((N - 256 wide_tiles) / 128)
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

// a stage holds the row blocks of A and 256 (128 with three row blocks) rows of B for one k-block
__host__ __device__ inline int b_boxes(int row_blocks) { return row_blocks <= 2 ? 2 : 1; }
__host__ __device__ inline int stage_bytes(int row_blocks) { return (row_blocks + b_boxes(row_blocks)) * kTileBytes; }
__host__ inline int ring_stages(int row_blocks) {
    const int s = (kSmemLimit - kAuxBytes) / stage_bytes(row_blocks);
    return s < kMaxStages ? s : kMaxStages;
}
__host__ inline int smem_bytes(int row_blocks) { return ring_stages(row_blocks) * stage_bytes(row_blocks) + kAuxBytes; }

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
gemm_umma_kernel(const GemmParams p, const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = smem_u32(smem);
    const int rb = p.row_blocks, stages = p.stages;
    const int sbytes = stage_bytes(rb);
    Aux* aux = reinterpret_cast<Aux*>(smem + stages * sbytes);
    volatile int* abort_flag = &aux->abort_flag;
    // may be launched as a programmatic dependent of the kernel before it in the stream
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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
        tma_prefetch_desc(&bmap);
    }
    if (warp == 0) { tmem_alloc(smem_u32(&aux->tmem_base), 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = aux->tmem_base;
    const int kblocks = p.K / kBK;
    const int wmax = b_boxes(rb) * kBN;            // widest tile: 256 columns, 128 with three row blocks
    const int nbuf = rb * wmax * 2 <= 512 ? 2 : 1; // accumulator buffers of rb x wmax columns each
    auto tile_col0 = [&](int tile) { return tile < p.wide_tiles ? tile * 2 * kBN : p.wide_tiles * 2 * kBN + (tile - p.wide_tiles) * kBN; };
    auto tile_width = [&](int tile) { return tile < p.wide_tiles ? 2 * kBN : kBN; };
    uint32_t issued = 0;

    if (warp == 0) {
        if (lane == 0) {
            const uint64_t stream_policy = l2_policy_evict_first();   // B is read once
            const uint64_t keep_policy = l2_policy_evict_last();      // A is read by every CTA for every tile
            uint32_t it = 0;
            for (int tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x) {
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t stage = it % stages, ph = (it / stages) & 1u;
                    if (!mbar_wait(smem_u32(&aux->empty[stage]), ph ^ 1u, abort_flag)) continue;
                    const uint32_t full = smem_u32(&aux->full[stage]);
                    const uint32_t dst = smem_base + stage * sbytes;
                    const int boxes = tile_width(tile) / kBN, col0 = tile_col0(tile);
                    mbar_arrive_expect_tx(full, (uint32_t)((rb + boxes) * kTileBytes));
                    for (int r = 0; r < rb; ++r) tma_load_2d_hint(dst + r * kTileBytes, &amap, full, kb * kBK, r * kBM, keep_policy);
                    for (int bx = 0; bx < boxes; ++bx)      // 128 rows of B each, back to back: one K-major operand of 256 rows
                        tma_load_2d_hint(dst + (rb + bx) * kTileBytes, &bmap, full, kb * kBK, col0 + bx * kBN, stream_policy);
                    issued = it + 1;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_128 = umma_idesc_16bit(kBM, kBN, 0, 0, false), idesc_256 = umma_idesc_16bit(kBM, 2 * kBN, 0, 0, false);
            uint32_t it = 0, tcount = 0;
            for (int tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x, ++tcount) {
                const uint32_t buf = tcount % nbuf, acc_ph = (tcount / nbuf) & 1u;
                const uint32_t idesc = tile_width(tile) == kBN ? idesc_128 : idesc_256;
                bool ok = mbar_wait(smem_u32(&aux->acc_empty[buf]), acc_ph ^ 1u, abort_flag);   // the epilogue has read this buffer
                tc_fence_after();
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t stage = it % stages, ph = (it / stages) & 1u;
                    ok = mbar_wait(smem_u32(&aux->full[stage]), ph, abort_flag) && ok;
                    tc_fence_after();
                    if (ok) {
                        const uint32_t a0 = smem_base + stage * sbytes;
                        const uint64_t bdesc = umma_smem_desc_sw128(a0 + rb * kTileBytes, 16, 1024);
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
        for (int tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x, ++tcount) {
            const uint32_t buf = tcount % nbuf, acc_ph = (tcount / nbuf) & 1u;
            const bool ok = mbar_wait(smem_u32(&aux->acc_full[buf]), acc_ph, abort_flag);
            tc_fence_after();
            const int n0 = tile_col0(tile), chunks = tile_width(tile) / 32;
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
                            if (col0 + j < p.N && (bi == 0xffffffffu || e > bv)) { bv = e; bi = (uint32_t)(col0 + j); }
                        }
                    } else {
                        float* dst = p.c + (long long)row * p.ldc + col0;
                        if (col0 + 32 <= p.N && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                reinterpret_cast<uint4*>(dst)[j] = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                        } else {
                            for (int j = 0; j < 32 && col0 + j < p.N; ++j) dst[j] = __uint_as_float(v[j]);
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

// Row-major bf16 matrix [rows, K] as a 2-D tensor map with boxes of 64 columns x 128 rows (128-byte swizzle): one box
// is one operand tile in the canonical K-major layout.  Rows past the end read as zeros.
inline int make_operand_map(EncodeTiledFn encode, CUtensorMap* map, const void* ptr, long long rows, long long K) {
    if (!encode) return -1;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {kBK, kBM};
    const cuuint32_t elem_strides[2] = {1, 1};
    return (int)encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, elem_strides,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// One sequence's acceptance walk per CTA over one key per row (the arg-max the product's epilogue left).
__global__ void __launch_bounds__(kArgmaxThreads) accept_walk_kernel(const AcceptParams p) {
    accept_walk_seq(p, (int)blockIdx.x);
}

}  // namespace gemm_path

// ------------------------------------------------------------------------------------------------------------
// The drafter cell's element-wise half (Eq. 2, 5-8): one CTA per row over the fp32 pre-activations
// S = h [W^f; W^i; W^o; W^c]^T ([rows, 4d]).  f = layer normalisation (biased variance, eps inside the root,
// optional affine) followed by exact GeLU.
// ------------------------------------------------------------------------------------------------------------
constexpr int kCellThreads = 1024;
constexpr int kCellPerThread = 16;               // d <= 16384

struct CellParams {
    const float* s;                  // [rows, 4d]
    const __nv_bfloat16* emb;        // [rows, d]  E(t), Eq. 1
    const float* gamma_c; const float* beta_c;   // affine of f in Eq. 6 (may be null)
    const float* gamma_z; const float* beta_z;   // affine of f in Eq. 8 (may be null)
    float* z;                        // [rows, d] in / out
    float* h_f32;                    // [rows, d] out (may be null)
    __nv_bfloat16* h_bf16;           // [rows, d] out (may be null)
    int d;
    float alpha, eps;
};

__device__ __forceinline__ float block_sum(float v, float* s_red) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();                 // s_red may still be read from the call before
    if (lane == 0) s_red[warp] = v;
    __syncthreads();
    float t = lane < kCellThreads / 32 ? s_red[lane] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    return t;
}

__device__ __forceinline__ float gelu_exact(float x) { return 0.5f * x * (1.f + erff(x * 0.70710678118654752f)); }
__device__ __forceinline__ float sigmoid_f(float x) { return 1.f / (1.f + __expf(-x)); }

__global__ void __launch_bounds__(kCellThreads) lstm_cell_kernel(const CellParams p) {
    __shared__ float s_red[kCellThreads / 32];
    const long long row = blockIdx.x;
    const int d = p.d;
    const float* s = p.s + row * 4ll * d;
    float xc[kCellPerThread], gi[kCellPerThread], zn[kCellPerThread];
    // s^c = W^c h + alpha e; its mean and variance over the d outputs (two passes over registers)
    float sum = 0.f;
#pragma unroll
    for (int k = 0; k < kCellPerThread; ++k) {
        const int j = k * kCellThreads + threadIdx.x;
        xc[k] = 0.f;
        if (j < d) { xc[k] = s[3ll * d + j] + p.alpha * __bfloat162float(p.emb[row * d + j]); sum += xc[k]; }
    }
    const float mean_c = block_sum(sum, s_red) / d;
    float sq = 0.f;
#pragma unroll
    for (int k = 0; k < kCellPerThread; ++k) {
        const int j = k * kCellThreads + threadIdx.x;
        if (j < d) { const float t = xc[k] - mean_c; sq += t * t; }
    }
    const float rstd_c = rsqrtf(block_sum(sq, s_red) / d + p.eps);
    // z' = z g^f + f(s^c) g^i  (Eq. 5-7)
    sum = 0.f;
#pragma unroll
    for (int k = 0; k < kCellPerThread; ++k) {
        const int j = k * kCellThreads + threadIdx.x;
        zn[k] = 0.f;
        if (j < d) {
            const float ae = p.alpha * __bfloat162float(p.emb[row * d + j]);
            float y = (xc[k] - mean_c) * rstd_c;
            if (p.gamma_c) y *= p.gamma_c[j];
            if (p.beta_c) y += p.beta_c[j];
            gi[k] = sigmoid_f(s[1ll * d + j] + ae);
            const float gf = sigmoid_f(s[j] + ae);
            zn[k] = p.z[row * d + j] * gf + gelu_exact(y) * gi[k];
            p.z[row * d + j] = zn[k];
            sum += zn[k];
        }
    }
    const float mean_z = block_sum(sum, s_red) / d;
    sq = 0.f;
#pragma unroll
    for (int k = 0; k < kCellPerThread; ++k) {
        const int j = k * kCellThreads + threadIdx.x;
        if (j < d) { const float t = zn[k] - mean_z; sq += t * t; }
    }
    const float rstd_z = rsqrtf(block_sum(sq, s_red) / d + p.eps);
    // h' = f(z') g^o  (Eq. 8)
#pragma unroll
    for (int k = 0; k < kCellPerThread; ++k) {
        const int j = k * kCellThreads + threadIdx.x;
        if (j < d) {
            float y = (zn[k] - mean_z) * rstd_z;
            if (p.gamma_z) y *= p.gamma_z[j];
            if (p.beta_z) y += p.beta_z[j];
            const float go = sigmoid_f(s[2ll * d + j] + p.alpha * __bfloat162float(p.emb[row * d + j]));
            const float h = gelu_exact(y) * go;
            if (p.h_f32) p.h_f32[row * d + j] = h;
            if (p.h_bf16) p.h_bf16[row * d + j] = __float2bfloat16_rn(h);
        }
    }
}

}  // namespace owl
