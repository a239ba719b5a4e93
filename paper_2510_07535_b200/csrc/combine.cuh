// LSE merge of the split-KV partials: for every output row whose keys were processed by more than
// one CTA, out = sum_s exp(lse_s - lse) o_s with lse = ln sum_s exp(lse_s); rounded to bf16.
// One warp per output row (packed node, query head); each lane owns 4 of the 128 output channels.
#pragma once

#include <cuda_fp16.h>

#include "owl_common.cuh"
#include "accept.cuh"

namespace owl {

constexpr int kCombineWarps = 8;

// One warp per output row finds the CTAs whose pieces cut the row's unit
// and merges their partials in CTA order.  A CTA stores at most two partials: slot 2c if its piece starts inside
// the unit, else 2c + 1.
//
// The kernel is launched as a programmatic dependent of that pass and its time after the pass has ended is pure
// latency, so everything that needs no output of the pass comes before the wait: for batches of at most 32
// sequences the warp derives the schedule from the inputs exactly as the pass did (warp_schedule) and knows its
// row's partial slots when the wait returns; what is left is one round of loads.  Larger batches read the
// schedule the pass left in global memory (first flat tile of every sequence, totals, choice of partition).
//
// kFused (verify step): the grid has one more CTA per sequence after the row CTAs; each of those runs one
// sequence's acceptance walk over the arg-max keys that the pass's spare warps left (`ap`).
//
// kGroup: partials fetched per round, 16 or 32.  A unit cut into 17 to 32 pieces (8 units of a 32K context over 148
// CTAs: 18 or 19) costs a second round of loads with 16, which is a whole memory round trip of a kernel that is
// all latency.  A round's rows go through a warp-private stage in shared memory (16 or 8 KB per warp: 128 or 64 KB
// per CTA, which is what limits 32 to launches with few rows; the host takes it up to 4096 output rows).
//
// The stage is there for the sake of the code's length, not of the data: with the rows in registers the fetch and
// the fold were two loops unrolled 32 times, some 450 instructions that a warp with one row executes exactly once,
// at the pace of instruction fetches from L2.  Copied with cp.async in a short rolled loop and folded in another,
// the same work is two dozen instructions executed from the instruction cache after their first trip (attention +
// merge call at 32K context 37.5 -> 36.8 us, with 8192 output rows 586 -> 578 us).
template <bool kFused, int kGroup>
__global__ void __launch_bounds__(kCombineWarps * 32) combine_sched_kernel(const AttnParams p, const AcceptParams ap) {
    const long long rows = (long long)p.total_nodes * p.num_q_heads;
    const unsigned row_ctas = (unsigned)p.combine_row_ctas;
    if (kFused) {
        if (blockIdx.x >= row_ctas) {
            static_assert(kCombineWarps * 32 >= kMaxNodes, "the walk needs one thread per node");
            asm volatile("griddepcontrol.wait;" ::: "memory");
            asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
            accept_walk_seq(ap, (int)(blockIdx.x - row_ctas));
            return;
        }
    }
    // The row CTAs are persistent: a warp derives the schedule once and then takes rows first, first + stride, ...
    // (one CTA per eight rows cost a launch of 8192 rows 19 us, most of it the schedule derived 8192 times).
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    extern __shared__ float4 combine_stage[];          // [warps][kGroup][32]: a round's partial rows, warp-private
    float4* stage = combine_stage + warp * kGroup * 32;
    const long long first = (long long)blockIdx.x * kCombineWarps + warp, stride = (long long)row_ctas * kCombineWarps;
    const bool small = p.batch <= 32;
    WarpSchedule ws{};
    Partition part;
    if (small) {
        ws = warp_schedule(p);
        part.init(ws.total, p.num_ctas, ws.units, ws.uniform_tiles);
    }
    // per row: its sequence, the CTAs c0..c1 whose pieces cut the row's unit, and the slot row of the partial this
    // lane fetches first
    int n = 0, hq = 0, b = 0, node_base = 0, tiles = 0, lrow = 0, c0 = 0, c1 = 0;
    long long seq_begin = 0, t0 = 0, prow_first = 0;
    auto row_of = [&](int c) -> long long { return (2ll * c + (part.begin(c) < t0 ? 1 : 0)) * p.rows_per_slot + lrow; };
    auto plan = [&]() {
        if (tiles == 0) return;
        const int G = p.group;
        lrow = (n - node_base) * G + hq % G;
        t0 = seq_begin + (long long)(hq / G) * tiles;
        c0 = part.owner(t0);
        c1 = part.owner(t0 + tiles - 1);
        prow_first = row_of(c0 + min(lane & (kGroup - 1), c1 - c0));
    };
    auto locate = [&](long long row_id) {       // every lane of the warp, same row
        n = (int)(row_id / p.num_q_heads);
        hq = (int)(row_id - (long long)n * p.num_q_heads);
        if (small) {
            const unsigned hit = __ballot_sync(0xffffffffu, lane < p.batch && ws.tiles > 0 && n >= ws.node_base && n < ws.node_base + ws.n);
            b = hit ? __ffs(hit) - 1 : 0;
            node_base = __shfl_sync(0xffffffffu, ws.node_base, b);
            tiles = hit ? __shfl_sync(0xffffffffu, ws.tiles, b) : 0;
            seq_begin = __shfl_sync(0xffffffffu, ws.excl_t, b);
        } else {
            int lo = 0, hi = p.batch;  // largest b with node_offsets[b] <= n
            if (p.node_offsets) {
                while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (p.node_offsets[mid] <= n) lo = mid; else hi = mid; }
                b = lo;
            } else {
                b = n / p.nodes_uniform;
            }
            const long long sb = p.sched_seq_begin[b], se = p.sched_seq_begin[b + 1];
            node_base = seq_node_base(p, b);
            seq_begin = sb;
            tiles = (int)((se - sb) / p.num_kv_heads);
        }
        plan();
    };
    // latency after the pass has ended is what this kernel costs: whatever needs no output of the pass comes before
    // the wait - for batches of at most 32 sequences the whole plan of the warp's first row
    if (small && first < rows) locate(first);
    // from here on the split-KV pass has completed and its writes are visible (a no-op in an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel in the stream may queue up
    if (!small) {
        const SchedHeader hdr = *p.sched_header;      // larger batches read the schedule the pass left
        part.init(hdr.total_tiles, p.num_ctas, hdr.units, hdr.uniform_tiles);
    }
    for (long long row_id = first; row_id < rows; row_id += stride) {
        if (!small || row_id != first) locate(row_id);
        if (tiles == 0) continue;
        if (c0 == c1) continue;  // a single CTA saw every key of this unit and wrote the result itself
        const int bad_epoch = __ldcg(p.seq_bad + b);   // (its round trip overlaps the partial loads below)
        const int count = c1 - c0 + 1;

        // Partials are taken kGroup at a time: lane j (< kGroup) of a group owns partial base + j.  The row loads do
        // not depend on the LSE values, so both go out together: one memory round trip per group.  Groups are folded
        // online (running maximum).
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float sum = 0.f, mx = -INFINITY;
        for (int base = 0; base < count; base += kGroup) {
            const int mine = base + (lane & (kGroup - 1));
            const bool have = mine < count;
            const long long prow = base == 0 ? prow_first : row_of(c0 + (have ? mine : 0));
            const float my_lse = have ? __ldcg(p.part_lse + prow) : -INFINITY;
            const int cnt = count - base < kGroup ? count - base : kGroup;
            if (base > 0) __syncwarp();                  // the stage's rows of the round before have been folded
#pragma unroll 1
            for (int j = 0; j < cnt; ++j) {
                const long long pj = __shfl_sync(0xffffffffu, prow, j);
                const uint32_t dst = (uint32_t)__cvta_generic_to_shared(stage + j * 32 + lane);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(p.part_o + pj * kHeadDim + lane * 4) : "memory");
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            float gmx = my_lse;
#pragma unroll
            for (int o = kGroup / 2; o > 0; o >>= 1) gmx = fmaxf(gmx, __shfl_xor_sync(0xffffffffu, gmx, o));
            const float mx_new = fmaxf(mx, gmx);
            if (mx_new > -INFINITY) {
                const float rescale = mx > -INFINITY ? __expf(mx - mx_new) : 0.f;
                acc.x *= rescale; acc.y *= rescale; acc.z *= rescale; acc.w *= rescale;
                sum *= rescale;
                const float w = have ? __expf(my_lse - mx_new) : 0.f;     // -inf partial: weight 0
                asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll 1
                for (int j = 0; j < cnt; ++j) {
                    const float wj = __shfl_sync(0xffffffffu, w, j);
                    const float4 v = stage[j * 32 + lane];                 // this lane's own copy: no barrier needed
                    acc.x += wj * v.x; acc.y += wj * v.y; acc.z += wj * v.z; acc.w += wj * v.w;
                    sum += wj;
                }
                mx = mx_new;
            } else {
                asm volatile("cp.async.wait_group 0;" ::: "memory");
            }
        }
        if (bad_epoch == p.epoch) continue;            // the pass found a bad tree or page in this sequence: no output
        const float inv = sum > 0.f ? 1.f / sum : 0.f;
        uint2 pk;
        if (p.f16) {
            __half2 lo2 = __floats2half2_rn(acc.x * inv, acc.y * inv), hi2 = __floats2half2_rn(acc.z * inv, acc.w * inv);
            pk.x = *reinterpret_cast<uint32_t*>(&lo2);
            pk.y = *reinterpret_cast<uint32_t*>(&hi2);
        } else {
            __nv_bfloat162 lo2 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), hi2 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
            pk.x = *reinterpret_cast<uint32_t*>(&lo2);
            pk.y = *reinterpret_cast<uint32_t*>(&hi2);
        }
        *reinterpret_cast<uint2*>(p.out + row_id * kHeadDim + lane * 4) = pk;
        if (p.lse && lane == 0) p.lse[row_id] = sum > 0.f ? mx + logf(sum) : -INFINITY;
    }
}

}  // namespace owl
