// The weight-streaming product of gemm_umma.cuh for 129 to 256 rows of A, on CTA pairs (cta_group::2).
//
// With two row blocks on one SM every k-step reads B's slice from shared memory twice (once per row block) and each
// k-block takes in 32 KB of A beside B's 28 KB: (4 x 22 KB read + 60 KB written) / 896 tensor clocks = 165 B per
// clock, above the 128 B per clock shared memory delivers - the launch was bound there, tensor pipe 68 % active.
// A pair of CTAs on neighbouring SMs runs one tcgen05.mma of M = 256 together: CTA r of the pair holds row block r
// of A, rows [r w/2, (r+1) w/2) of the tile's B and its own 128 rows of the accumulator, so per SM a k-step reads
// 4 KB + w/64 KB and a k-block writes 16 KB + w/16 KB: 134 B per clock at w = 224.  Each SM's tensor memory now
// holds two accumulator buffers of 256 columns, so the epilogue of a tile hides under the next tile's products
// (one CTA with two row blocks had room for a single buffer).
// One thread issues for two SMs, and what it does between two batches of products (a wait, a commit) is not hidden
// behind them: with one k-block per stage - four products of 112 clocks between a wait and a commit - the pair was no
// faster than two single CTAs (5-8 % slower under the power cap).  A stage therefore holds TWO k-blocks (60 KB at
// w = 224, three stages): eight products per wait and commit.  128256 columns x 4096, bf16: 256 rows 244 -> 209 us,
// 192 rows 235 -> 205 us, 160 rows 226 -> 203 us against the single-CTA kernel (same-process A/B, best of 31 regions
// each; medians 296 -> 235 us at 256 rows), 1287 TFLOP/s.  K must be a multiple of 128; other shapes take the
// single-CTA kernel.
//
// Roles per CTA (256 threads):
//   warp 0     TMA producer: its half of every k-block into its own ring; the copies complete on the EVEN CTA's
//              arrival barrier (a .cta_group::2 copy may name a barrier of the peer CTA; no multicast anywhere)
//   warp 1     even CTA only: issues the pair's tcgen05.mma (one thread) and the commits, which arrive on the
//              barriers of both CTAs
//   warps 4-7  epilogue of the CTA's own 128 rows, as in the single-CTA kernel
// Every wait is bounded; a wait that gives up raises the abort flag of both CTAs.
#pragma once

#include "gemm_umma.cuh"

namespace owl {
namespace gemm_path {

struct PairAux {
    uint64_t full[kMaxStages], empty[kMaxStages];   // `full` is used in the even CTA only
    uint64_t acc_full[2], acc_empty[2];             // `acc_empty` is used in the even CTA only (256 arrivals)
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(PairAux) <= kAuxBytes, "aux area too small");

// .cta_group::2 form of the tile copy: destination in this CTA, completion counted on `bar_cluster`, a
// shared::cluster address that may lie in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const void* tmap, uint32_t bar_cluster, int c0, int c1, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        : : "r"(dst), "l"(tmap), "r"(bar_cluster), "r"(c0), "r"(c1), "l"(policy) : "memory");
}

// p.row_blocks == 2; p.w_lo and the round widths are whole-tile widths (each CTA stages half of a tile's rows of B:
// the boxes of bmap_hi / bmap_lo are (w_lo + 16) / 2 and w_lo / 2 rows high); p.a_bytes = 16 KB; p.stage_bytes =
// 2 x (16 KB + half of the widest tile's rows of B), the two k-blocks of a stage one after the other; K % 128 == 0.
// gridDim.x is even: CTAs 2j and 2j + 1 are pair j.
template <int kEpi>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_umma_pair_kernel(const GemmParams p, const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap bmap_hi,
                      const __grid_constant__ CUtensorMap bmap_lo) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t ring = smem_u32(smem) + kAuxBytes;
    const int stages = p.stages, sbytes = p.stage_bytes;
    PairAux* aux = reinterpret_cast<PairAux*>(smem);
    volatile int* abort_flag = &aux->abort_flag;
    const uint32_t rank = cluster_cta_rank();           // 0: issues the products; 1: its peer
    const int pair = (int)(blockIdx.x >> 1), pairs = (int)(gridDim.x >> 1);
    // the peer's abort flag: a wait that gives up here ends the peer's waits too
    const uint32_t peer_abort = cluster_map(smem_u32(&aux->abort_flag), rank ^ 1u);
    auto wait = [&](uint32_t bar, uint32_t parity) {
        const bool ok = mbar_wait_cluster_ns(bar, parity, abort_flag, kWaitLimitNs);
        if (!ok) st_cluster_u32(peer_abort, 1u);
        return ok;
    };
    const bool misaligned = (ring & 1023u) != 0;       // operand tiles must sit on swizzle-atom boundaries (same in both CTAs)
    if (tid == 0) {
        for (int i = 0; i < stages; ++i) { mbar_init(smem_u32(&aux->full[i]), 1); mbar_init(smem_u32(&aux->empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&aux->acc_full[i]), 1); mbar_init(smem_u32(&aux->acc_empty[i]), 256); }
        aux->abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&amap);
        tma_prefetch_desc(&bmap_hi);
        tma_prefetch_desc(&bmap_lo);
    }
    if (warp == 0 && !misaligned) { tmem_alloc_pair(smem_u32(&aux->tmem_base), 512); tmem_relinquish_pair(); }
    // may be launched as a programmatic dependent: the set-up above touched no input
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    tc_fence_before();
    cluster_sync_all();            // both CTAs' barriers are initialised and both halves of tensor memory allocated
    tc_fence_after();
    if (misaligned) {
        if (tid == 0) report(p.status, kErrTimeout);
        return;
    }
    const uint32_t tmem = aux->tmem_base;
    const int kblocks = p.K / kBK;
    auto tile_width = [&](int t) { return t < p.wide_rounds ? p.w_lo + 16 : p.w_lo; };
    auto tile_col0 = [&](int t) {
        const int hi = t < p.wide_rounds ? t : p.wide_rounds;
        return pairs * (hi * (p.w_lo + 16) + (t - hi) * p.w_lo) + pair * tile_width(t);
    };
    uint32_t issued = 0;

    if (warp == 0) {
        if (lane == 0) {
            const uint64_t stream_policy = l2_policy_evict_first();   // B is read once
            const uint64_t keep_policy = l2_policy_evict_last();      // A is read by every pair for every tile
            uint32_t it = 0;
            for (int t = 0; t < p.rounds; ++t) {
                const int col0 = tile_col0(t), half = tile_width(t) >> 1;
                if (col0 >= p.N) break;
                const CUtensorMap* bmap = t < p.wide_rounds ? &bmap_hi : &bmap_lo;   // box = half of the tile's rows of B
                for (int kb = 0; kb < kblocks; kb += 2, ++it) {     // a stage holds two k-blocks (K is a multiple of 128)
                    const uint32_t stage = it % stages, ph = (it / stages) & 1u;
                    if (!wait(smem_u32(&aux->empty[stage]), ph ^ 1u)) continue;
                    // both CTAs' copies of this stage complete on the even CTA's barrier, which expects all their bytes
                    const uint32_t full0 = cluster_map(smem_u32(&aux->full[stage]), 0);
                    const uint32_t dst = ring + stage * sbytes;
                    if (rank == 0) mbar_arrive_expect_tx(smem_u32(&aux->full[stage]), 4u * (uint32_t)(kTileBytes + half * kBK * 2));
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        tma_load_2d_pair(dst + q * (sbytes >> 1), &amap, full0, (kb + q) * kBK, (int)rank * kBM, keep_policy);
                        tma_load_2d_pair(dst + q * (sbytes >> 1) + kTileBytes, bmap, full0, (kb + q) * kBK, col0 + (int)rank * half, stream_policy);
                    }
                    issued = it + 1;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, tcount = 0;
            for (int t = 0; t < p.rounds; ++t, ++tcount) {
                if (tile_col0(t) >= p.N) break;
                const uint32_t buf = tcount & 1u, acc_ph = (tcount >> 1) & 1u;
                const uint32_t idesc = umma_idesc_16bit(2 * kBM, tile_width(t), 0, 0, false);
                bool ok = wait(smem_u32(&aux->acc_empty[buf]), acc_ph ^ 1u);      // both epilogues have read this buffer
                tc_fence_after();
                for (int kb = 0; kb < kblocks; kb += 2, ++it) {
                    const uint32_t stage = it % stages, ph = (it / stages) & 1u;
                    ok = wait(smem_u32(&aux->full[stage]), ph) && ok;
                    tc_fence_after();
                    if (ok) {
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const uint32_t a0 = ring + stage * sbytes + q * (sbytes >> 1);
                            const uint64_t adesc = umma_smem_desc_sw128(a0, 16, 1024);
                            const uint64_t bdesc = umma_smem_desc_sw128(a0 + kTileBytes, 16, 1024);
#pragma unroll
                            for (int ks = 0; ks < kBK / 16; ++ks)
                                umma_ss_pair(tmem + buf * 256u, adesc + (uint64_t)(ks * 2), bdesc + (uint64_t)(ks * 2), idesc, (kb | q | ks) ? 1u : 0u);
                        }
                        umma_commit_pair(smem_u32(&aux->empty[stage]), 3);       // the slot is free in both CTAs
                    }
                }
                if (ok) umma_commit_pair(smem_u32(&aux->acc_full[buf]), 3);
            }
        }
    } else if (warp >= 4) {
        const int lane_row = (warp & 3) * 32 + lane;                    // TMEM lane = row inside the CTA's row block
        const uint32_t lane_sel = (uint32_t)((warp & 3) * 32) << 16;
        const int row = (int)rank * kBM + lane_row;
        uint32_t tcount = 0;
        for (int t = 0; t < p.rounds; ++t, ++tcount) {
            const int n0 = tile_col0(t);
            if (n0 >= p.N) break;
            const uint32_t buf = tcount & 1u, acc_ph = (tcount >> 1) & 1u;
            const bool ok = wait(smem_u32(&aux->acc_full[buf]), acc_ph);
            tc_fence_after();
            const int n_end = n0 + tile_width(t) < p.N ? n0 + tile_width(t) : p.N;
            const int chunks = (tile_width(t) + 31) / 32;
            const uint32_t taddr = tmem + lane_sel + buf * 256u;
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
            tc_fence_before();
            // unconditional: the issuing thread's wait on the even CTA's barrier must end
            mbar_arrive_cluster(cluster_map(smem_u32(&aux->acc_empty[buf]), 0));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (aux->abort_flag && warp == 0 && lane == 0) {
        if (rank == 0) {
            // both CTAs' copies complete on this CTA's barriers: give those in flight a bounded time to land before
            // either CTA's shared memory is released (the peer leaves only after the cluster barrier below)
            const uint32_t first = issued > (uint32_t)stages ? issued - stages : 0u;
            for (uint32_t it = first; it < issued; ++it) {
                const uint32_t bar = smem_u32(&aux->full[it % stages]), ph = (it / stages) & 1u;
                for (int polls = 0; polls < (1 << 20) && !mbar_try_wait_cluster(bar, ph); ++polls) {}
            }
        }
        report(p.status, kErrTimeout);
    }
    // no CTA leaves while its peer may still send it an arrival or read or write its half of a product
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc_pair(tmem, 512);
    }
}

}  // namespace gemm_path
}  // namespace owl
