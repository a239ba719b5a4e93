// Split-KV verify attention on the 5th-generation tensor cores (tcgen05.mma, accumulators in
// tensor memory), K/V tiles staged by TMA.
//
// One persistent CTA per SM, 12 warps:
//   warp 0        TMA producer: per 128-key tile, one box per (page, head) for K and for V into a
//                 ring of 32 KB shared-memory slots (layout in kv_tensor_map.cuh)
//   warp 1        issues every tcgen05.mma (one lane) and the commits that signal their completion
//   warps 2-3     no part in the attention; in a verify step with a small logits scan they do that scan
//   warps 4-7     softmax warpgroup of stream 0   (one thread per packed row)
//   warps 8-11    softmax warpgroup of stream 1
// A unit is one (sequence, KV head) with M = G * n packed rows (row = node * G + head in group).
// The two streams are two independent online-softmax pipelines, each with its own score tile S
// (128 x 128 fp32, columns of tensor memory), its own bf16 probabilities P (written over S) and its
// own output accumulator O (128 x 128 fp32):
//   M > 128  ("shared"): stream s owns rows [128 s, 128 s + 128); both streams consume every K/V tile,
//            which is therefore read from HBM and staged once for all 256 rows;
//   M <= 128 ("split"):  both streams hold the same rows; stream s consumes the key tiles of parity s,
//            and the two partial results are merged by their log-sum-exp when the segment ends.
// Either way the tensor pipe always has the other stream's products to run while one stream's
// warpgroup is in its softmax.  Per tile and stream: S = Q K^T (8 MMAs of K = 16 over the head
// dimension), softmax warpgroup reads S, applies the tree mask on the few tiles that reach drafted
// positions, updates the running maximum lazily (O is rescaled only when the maximum grew by more
// than 2^8), writes P, then O += P V (8 MMAs over the keys, A operand from tensor memory, V as an
// MN-major B operand).
//
// Work is cut as in owl_common.cuh (flat range of 128-key tiles over all units, equal pieces per
// CTA); a CTA whose piece covers a whole unit writes the final bf16 output, otherwise a normalised
// fp32 partial and its LSE for the combine kernel.
//
// Every mbarrier wait is bounded (sm100_ptx.cuh).  When a wait gives up, the CTA's abort flag makes
// all later waits return at once, MMA issue and output writes stop, the loops run out (they are
// finite), the producer waits - bounded - for its TMA copies in flight, tensor memory is freed and
// the status word reports OWL_ERR_TIMEOUT.
#pragma once

#include <cuda_fp16.h>

#include <type_traits>

#include "kv_tensor_map.cuh"
#include "owl_common.cuh"
#include "accept.cuh"
#include "sm100_ptx.cuh"

namespace owl {
namespace umma_path {

using namespace sm100;

constexpr int kTileKeys = 128;
constexpr int kRows = 256;                 // packed rows per unit (two streams of 128)
constexpr int kThreads = 384;
constexpr int kSlots = 5;                  // ring of K / V tiles
constexpr int kSlotBytes = kTileKeys * kHeadDim * 2;     // 32 KB
constexpr int kTilesInFlight = 3;          // five slots never hold parts of more than three tiles
constexpr int kQBytes = 128 * kHeadDim * 2;              // 32 KB per 128-row block
constexpr int kRingOff = 2 * kQBytes;
constexpr int kAuxOff = kRingOff + kSlots * kSlotBytes;  // 224 KB
constexpr int kAuxBytes = 3072;
constexpr int kSmemBytes = kAuxOff + kAuxBytes;          // 232448 = 227 KB
constexpr uint32_t kTmemCols = 512;
constexpr float kLazyRescale = 8.0f;       // log2 units

struct Aux {
    uint64_t full[kTilesInFlight];   // one per tile: its K and its V slot complete the same barrier
    uint64_t empty[kSlots];
    uint64_t s_full[2], o_done[2];
    uint64_t q_full;
    uint32_t tmem_base;
    int abort_flag;
    int seg_bad_tree;
    int sched_b0;
    long long sched_tile_begin;
    long long scan_tiles[12];
    long long total_tiles;
    int scan_units[12];
    int scan_tmin[12], scan_tmax[12];
    int sched_unit_begin;
    short parent[kMaxNodes];
    unsigned long long anc[kMaxNodes];
};
static_assert(sizeof(Aux) <= kAuxBytes, "aux area too small");

struct Segment {
    int b, h, unit, n, L, node_base, M;
    int tiles, tile0, tile1;
    bool shared;
    __device__ __forceinline__ int iters(int s) const {
        const int T = tile1 - tile0;
        return shared ? T : (s == 0 ? (T + 1) >> 1 : T >> 1);
    }
    __device__ __forceinline__ int tile(int s, int i) const { return tile0 + (shared ? i : 2 * i + s); }
    __device__ __forceinline__ bool whole() const { return tile0 == 0 && tile1 == tiles; }
};

// Walks the CTA's piece [t, t_end) of the flat tile range unit by unit.  Every role runs its own
// copy; all copies see the same sequence of segments.
struct Walker {
    int b, unit_begin;
    long long seq_begin, t, t_end;
    // the sequence `b` as last loaded (most segments of a piece lie in the same sequence)
    int cur_b = -1, cur_n = 0, cur_L = 0, cur_tiles = 0, cur_node_base = 0;
    bool cur_ok = false;
    __device__ __forceinline__ void load_seq(const AttnParams& p) {
        cur_n = seq_nodes(p, b);
        cur_L = p.ctx_lens[b];
        cur_ok = seq_shape_ok(p, b, cur_n, cur_L);
        cur_tiles = cur_ok ? (cur_L + cur_n + kTileKeys - 1) / kTileKeys : 0;
        cur_node_base = seq_node_base(p, b);
        cur_b = b;
    }
    // kWide = false: the caller knows that no unit has more than 128 rows (G * max_nodes <= 128, and sequences with
    // more nodes than max_nodes are rejected), so `shared` is a constant and the code of that mode is not generated.
    template <bool kWide>
    __device__ __forceinline__ bool next(const AttnParams& p, Segment& g) {
        if (t >= t_end) return false;
        while (b < p.batch) {
            if (cur_b != b) load_seq(p);
            const long long flat = (long long)cur_tiles * p.num_kv_heads;
            if (t < seq_begin + flat) break;
            seq_begin += flat;
            unit_begin += cur_ok ? p.num_kv_heads : 0;
            ++b;
        }
        if (b >= p.batch) { t = t_end; return false; }
        const int tiles = cur_tiles;
        const unsigned local = (unsigned)(t - seq_begin);   // < tiles * Hkv <= 2^24 * 2^7
        g.b = b; g.n = cur_n; g.L = cur_L; g.tiles = tiles;
        g.h = (int)(local / (unsigned)tiles);
        g.tile0 = (int)(local - (unsigned)g.h * (unsigned)tiles);
        const long long left = t_end - t;
        g.tile1 = (int)(g.tile0 + left < tiles ? g.tile0 + left : tiles);
        g.unit = unit_begin + g.h;
        g.node_base = cur_node_base;
        g.M = cur_n * p.group;
        g.shared = kWide && g.M > 128;
        t += g.tile1 - g.tile0;
        return true;
    }
};

// Block-wide: totals of the flat tile range, the choice of partition and the first sequence of this
// CTA's piece.  CTA 0 also leaves the per-sequence prefix and the header for the combine kernel.
__device__ __forceinline__ void build_walk(const AttnParams& p, Aux* aux, Walker& w) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int per = (p.batch + kThreads - 1) / kThreads;
    const int b_lo = tid * per, b_hi = min(p.batch, b_lo + per);
    long long my_tiles = 0;
    int my_units = 0, tmin = 0x7fffffff, tmax = 0;
    for (int b = b_lo; b < b_hi; ++b) {
        const int n = seq_nodes(p, b), L = p.ctx_lens[b];
        if (seq_shape_ok(p, b, n, L)) {
            const int tiles = (L + n + kTileKeys - 1) / kTileKeys;
            my_tiles += (long long)tiles * p.num_kv_heads;
            my_units += p.num_kv_heads;
            tmin = min(tmin, tiles); tmax = max(tmax, tiles);
        } else {
            report(p.status, seq_tree_shape_ok(p, b, n) ? kErrBadPage : kErrBadTree);
            p.seq_bad[b] = p.epoch;
        }
    }
    long long inc_t = my_tiles;
    int inc_u = my_units;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const long long vt = __shfl_up_sync(0xffffffffu, inc_t, o);
        const int vu = __shfl_up_sync(0xffffffffu, inc_u, o);
        if (lane >= o) { inc_t += vt; inc_u += vu; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        tmin = min(tmin, __shfl_xor_sync(0xffffffffu, tmin, o));
        tmax = max(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
    }
    if (lane == 31) { aux->scan_tiles[warp] = inc_t; aux->scan_units[warp] = inc_u; aux->scan_tmin[warp] = tmin; aux->scan_tmax[warp] = tmax; }
    __syncthreads();
    long long off_t = 0, total = 0;
    int off_u = 0, units = 0;
#pragma unroll 1
    for (int w2 = 0; w2 < kThreads / 32; ++w2) {
        if (w2 < warp) { off_t += aux->scan_tiles[w2]; off_u += aux->scan_units[w2]; }
        total += aux->scan_tiles[w2]; units += aux->scan_units[w2];
        tmin = min(tmin, aux->scan_tmin[w2]); tmax = max(tmax, aux->scan_tmax[w2]);
    }
    const int uniform_tiles = (units > 0 && tmin == tmax) ? tmin : 0;
    const long long excl_t = off_t + inc_t - my_tiles;
    const int excl_u = off_u + inc_u - my_units;
    Partition part;
    part.init(total, gridDim.x, units, uniform_tiles);
    long long t_begin, t_end;
    part.range(blockIdx.x, t_begin, t_end);
    if (t_begin < t_end && my_tiles > 0 && t_begin >= excl_t && t_begin < excl_t + my_tiles) {
        aux->sched_b0 = b_lo;                 // the walker skips ahead from the first sequence of this thread
        aux->sched_tile_begin = excl_t;
        aux->sched_unit_begin = excl_u;
    }
    if (blockIdx.x == 0) {
        long long run = excl_t;
        for (int b = b_lo; b < b_hi; ++b) {
            p.sched_seq_begin[b] = run;
            const int n = seq_nodes(p, b), L = p.ctx_lens[b];
            if (seq_shape_ok(p, b, n, L)) run += (long long)((L + n + kTileKeys - 1) / kTileKeys) * p.num_kv_heads;
        }
        if (tid == 0) {
            p.sched_seq_begin[p.batch] = total;
            p.sched_header->total_tiles = total;
            p.sched_header->uniform_tiles = uniform_tiles;
            p.sched_header->units = units;
        }
    }
    __syncthreads();
    w.t = t_begin;
    w.t_end = t_end;
    w.b = aux->sched_b0;
    w.seq_begin = aux->sched_tile_begin;
    w.unit_begin = aux->sched_unit_begin;
}

// Batches of at most 32 sequences: every warp derives the same schedule on its own (lane b holds sequence
// b, prefix sums by shuffle), with no shared memory and no CTA-wide barrier, so that each role can start
// as soon as its own loads have returned.
__device__ __forceinline__ void build_walk_small(const AttnParams& p, Walker& w) {
    static_assert(kTileKeys == kSchedTileKeys, "the merge kernel derives the same schedule");
    const int lane = threadIdx.x & 31;
    const WarpSchedule ws = warp_schedule(p);
    const int n = ws.n, L = ws.L, node_base = ws.node_base, tiles = ws.tiles;
    if (lane < p.batch && !ws.ok && threadIdx.x < 32) {
        report(p.status, seq_tree_shape_ok(p, lane, n) ? kErrBadPage : kErrBadTree);
        p.seq_bad[lane] = p.epoch;
    }
    const long long my_tiles = ws.my_tiles, total = ws.total, excl_t = ws.excl_t;
    const int units = ws.units, uniform_tiles = ws.uniform_tiles, excl_u = ws.excl_u;
    Partition part;
    part.init(total, gridDim.x, units, uniform_tiles);
    long long t_begin, t_end;
    part.range(blockIdx.x, t_begin, t_end);
    const unsigned owner = __ballot_sync(0xffffffffu, my_tiles > 0 && t_begin >= excl_t && t_begin < excl_t + my_tiles);
    if (blockIdx.x == 0 && threadIdx.x < 32) {
        if (lane < p.batch) p.sched_seq_begin[lane] = excl_t;
        if (lane == 0) {
            p.sched_seq_begin[p.batch] = total;
            p.sched_header->total_tiles = total;
            p.sched_header->uniform_tiles = uniform_tiles;
            p.sched_header->units = units;
        }
    }
    w.t = t_begin;
    w.t_end = (t_begin < t_end && owner) ? t_end : t_begin;
    const int b0 = owner ? __ffs(owner) - 1 : 0;
    w.b = b0;
    w.seq_begin = __shfl_sync(0xffffffffu, excl_t, b0);
    w.unit_begin = __shfl_sync(0xffffffffu, excl_u, b0);
    w.cur_b = b0;
    w.cur_n = __shfl_sync(0xffffffffu, n, b0);
    w.cur_L = __shfl_sync(0xffffffffu, L, b0);
    w.cur_node_base = __shfl_sync(0xffffffffu, node_base, b0);
    w.cur_tiles = __shfl_sync(0xffffffffu, tiles, b0);
    w.cur_ok = true;
}

// ------------------------------------------------------------------------------------------ producer
template <bool kWide>
__device__ __forceinline__ void producer_loop(const AttnParams& p, const CUtensorMap* kmap, const CUtensorMap* vmap,
                                              Aux* aux, uint32_t ring, Walker w, uint32_t& items_out) {
    const int lane = threadIdx.x & 31;
    volatile int* abort_flag = &aux->abort_flag;
    const int ppt = kTileKeys >> p.page_shift;               // pages (= TMA boxes) per tile
    const uint32_t box_bytes = (uint32_t)p.page_size * 256u;
    const int oob = p.num_pages * p.num_kv_heads;            // a coordinate past the end: the box reads zeros
    uint32_t item = 0;
    // K/V are read once: let them leave L2 first, so that Q, the partials, the tables and the code stay
    const uint64_t stream_policy = l2_policy_evict_first();
    Segment g;
    while (w.template next<kWide>(p, g)) {
        const int keys = g.L + g.n;
        const int pages_valid = (keys + p.page_size - 1) >> p.page_shift;
        const int32_t* table = p.block_table + (long long)g.b * p.max_pages_per_seq;
        auto coord_of = [&](int t) {
            int c = oob;
            const int lp = t * ppt + lane;
            if (lane < ppt && lp < pages_valid) {
                const int pg = table[lp];
                if ((unsigned)pg < (unsigned)p.num_pages) c = pg * p.num_kv_heads + g.h;
                else { report(p.status, kErrBadPage); p.seq_bad[g.b] = p.epoch; }
            }
            return c;
        };
        int c_next = coord_of(g.tile0);
        for (int t = g.tile0; t < g.tile1; ++t) {
            const int c_cur = c_next;
            if (t + 1 < g.tile1) c_next = coord_of(t + 1);
#pragma unroll
            for (int kv = 0; kv < 2; ++kv) {
                const uint32_t slot = item % kSlots, ph = (item / kSlots) & 1u;
                const uint32_t full = smem_u32(&aux->full[(item >> 1) % kTilesInFlight]);
                const bool ok = mbar_wait(smem_u32(&aux->empty[slot]), ph ^ 1u, abort_flag);
                if (ok) {
                    // the tile's barrier expects K and V together (announced with K; V follows as its slot frees up)
                    if (lane == 0 && kv == 0) mbar_arrive_expect_tx(full, 2u * (uint32_t)kSlotBytes);
                    __syncwarp();
                    if (lane < ppt)
                        tma_load_5d_hint(ring + slot * kSlotBytes + lane * box_bytes, kv ? vmap : kmap, full, 0, 0, 0, 0, c_cur,
                                         stream_policy);
                    ++item;
                }
                __syncwarp();
            }
        }
    }
    items_out = item;
}

// ------------------------------------------------------------------------------------------ MMA issuer
// One thread's time is what bounds a 256-row unit: each tcgen05.mma costs the issuing thread about 60 clocks, and
// whatever it executes between two batches (waits, slot arithmetic, commits) is added to that, not hidden behind it.
// So the loop is kept lean:
//  * the warp stays converged from top to bottom; all 32 lanes run the loop and the tensor-core instructions carry
//    the guard (`elected` lane, waits succeeded, work to do) themselves.  What steers the loop (the segment's tile
//    range and mode, the verdicts of the waits) goes through a warp reduction or a vote first, so that trip counts,
//    ring slots and descriptors are uniform by construction;
//  * per tile of such a unit it waits on hardware barriers only (about 25 clocks each when the arrival is already
//    in; a look at an mbarrier costs 70 to 130): one per stream, on which the softmax warpgroup announces P, and
//    one on which stream 0's warpgroup tells that it has seen the next key tile arrive (units of up to 128 rows
//    wait for the tile itself);
//  * the iterations in which both streams have both products to issue run in a loop of their own without
//    per-product conditions; the first and the last ones of a segment take the general form.
template <bool kWide, bool kF16>
__device__ __forceinline__ void mma_loop(const AttnParams& p, Aux* aux, uint32_t smem_base, uint32_t tmem, Walker w) {
    constexpr unsigned kAll = 0xffffffffu;
    volatile int* abort_flag = &aux->abort_flag;
    constexpr uint32_t idesc_qk = umma_idesc_16bit(128, kTileKeys, 0, 0, kF16);
    constexpr uint32_t idesc_pv = umma_idesc_16bit(128, kHeadDim, 0, 1, kF16);
    const uint32_t ring = smem_base + kRingOff;
    const uint32_t elected = elect_one() ? 1u : 0u;
    // descriptors of Q block 0 and of ring slot 0; those of the other blocks and slots differ in the start-address
    // field only (units of 16 bytes; shared memory ends below 2^18, so the field never carries)
    const uint64_t q_desc0 = umma_smem_desc_sw128(smem_base, 16, 1024);
    const uint64_t k_desc0 = umma_smem_desc_sw128(ring, 16, 2048), v_desc0 = umma_smem_desc_sw128(ring, 1024, 2048);
    uint32_t seg_no = 0, item_base = 0;
    Segment g;

    for (;;) {
        const bool more = w.template next<kWide>(p, g);
        if (!__any_sync(kAll, more)) break;
        const int tile0 = __reduce_max_sync(kAll, g.tile0), tile1 = __reduce_max_sync(kAll, g.tile1);
        const bool shared = kWide && __reduce_max_sync(kAll, g.shared ? 1 : 0) != 0;
        bool ok = __all_sync(kAll, mbar_wait(smem_u32(&aux->q_full), seg_no & 1u, abort_flag));
        const int T = tile1 - tile0;
        const int n_it[2] = {shared ? T : (T + 1) >> 1, shared ? T : T >> 1};

        // ring slots of the K tile and of the V tile each stream needs next, as running counters
        const uint32_t step_items = shared ? 2u : 4u;
        uint32_t k_slot[2], v_slot[2];
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const uint32_t first = item_base + (shared ? 0u : 2u * (uint32_t)s);
            k_slot[s] = first % kSlots;
            v_slot[s] = (first + 1u) % kSlots;
        }
        auto advance = [&](uint32_t& slot) { slot += step_items; if (slot >= (uint32_t)kSlots) slot -= kSlots; };
        // O_s (+)= P_s V: A from tensor memory, B = the V tile as it lies in the ring (MN-major)
        auto issue_pv = [&](int s, uint32_t issue, uint32_t acc0) {
            const uint32_t v_lo = (uint32_t)v_desc0 + v_slot[s] * (uint32_t)(kSlotBytes >> 4), v_hi = (uint32_t)(v_desc0 >> 32);
            const uint32_t tO = tmem + 256 + s * 128, tP = tmem + s * 128;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                umma_ts_lh_if(issue, tO, tP + ks * 8, v_lo + (uint32_t)(ks * 4096 >> 4), v_hi, idesc_pv, ks ? 1u : acc0);
        };
        // S_s = Q K^T: both operands K-major in shared memory
        auto issue_qk = [&](int s, uint32_t issue) {
            const uint32_t q_lo = (uint32_t)q_desc0 + (uint32_t)((shared && s) ? (kQBytes >> 4) : 0), q_hi = (uint32_t)(q_desc0 >> 32);
            const uint32_t k_lo = (uint32_t)k_desc0 + k_slot[s] * (uint32_t)(kSlotBytes >> 4), k_hi = (uint32_t)(k_desc0 >> 32);
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_ss_lh_if(issue, tmem + s * 128, q_lo + (uint32_t)((hf * 16384 + ks * 32) >> 4), q_hi,
                                  k_lo + (uint32_t)((hf * 1024 + ks * 32) >> 4), k_hi, idesc_qk, (hf | ks) ? 1u : 0u);
        };
        // Before S = Q K^T of the stream's tile i + 1.  M > 128: the issue loop is what bounds the unit, and the
        // softmax warpgroup, which has time to spare, looks at the tile's arrival barrier and passes the news on
        // through hardware barrier 6 (about 25 clocks here).  M <= 128: the tile itself is what the warp
        // usually waits for, and it waits on the arrival barrier directly, one wake-up instead of two.
        auto wait_next_k = [&](int s, int i) {
            if (shared) {
                // (both streams read the tile: stream 1 finds what stream 0 has just made sure of)
                if (s == 0) asm volatile("bar.sync 6, 64;" ::: "memory");
            } else {
                const uint32_t seq = (item_base >> 1) + (uint32_t)(2 * (i + 1) + s);
                ok = __all_sync(kAll, mbar_wait(smem_u32(&aux->full[seq % kTilesInFlight]), (seq / kTilesInFlight) & 1u,
                                                abort_flag)) && ok;
            }
        };
        // The same two products with the k-steps in a loop, for the few iterations of the general form below (they
        // are too rare to be worth the code size of another thirty-two unrolled instructions)
        auto issue_pv_rolled = [&](int s, uint32_t issue, uint32_t acc0) {
            uint64_t vdesc = v_desc0 + (uint64_t)(v_slot[s] * (uint32_t)(kSlotBytes >> 4));
            const uint32_t tO = tmem + 256 + s * 128;
            uint32_t tP = tmem + s * 128;
#pragma unroll 1
            for (int ks = 0; ks < 8; ++ks, vdesc += 4096 >> 4, tP += 8)
                umma_ts_if(issue, tO, tP, vdesc, idesc_pv, ks ? 1u : acc0);
        };
        auto issue_qk_rolled = [&](int s, uint32_t issue) {
            uint64_t qdesc = q_desc0 + (uint64_t)((shared && s) ? (kQBytes >> 4) : 0);
            uint64_t kdesc = k_desc0 + (uint64_t)(k_slot[s] * (uint32_t)(kSlotBytes >> 4));
#pragma unroll 1
            for (int j = 0; j < 8; ++j) {
                umma_ss_if(issue, tmem + s * 128, qdesc, kdesc, idesc_qk, j ? 1u : 0u);
                // four k-steps of 32 bytes inside a 128-byte swizzle row, then the other half of the head dimension
                qdesc += j == 3 ? (uint64_t)((16384 - 96) >> 4) : 2u;
                kdesc += j == 3 ? (uint64_t)((1024 - 96) >> 4) : 2u;
            }
        };
        // General form of one iteration: O += P V of tile i, then S = Q K^T of tile i + 1 (which overwrites the P just
        // consumed; the tensor pipe runs them in order), each where the stream has such a tile.  i = -1 issues the
        // first S of both streams, after this warp's own look at the arrival barrier of their first tiles.
        auto general = [&](int i) {
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                const bool last_reader = !shared || s == 1;
                const bool do_pv = i >= 0 && i < n_it[s], do_qk = i + 1 < n_it[s];
                if (do_pv) asm volatile("bar.sync %0, 160;" ::"r"(4 + s) : "memory");
                if (i < 0 && do_qk && !(shared && s == 1)) {
                    const uint32_t seq = (item_base >> 1) + (uint32_t)s;
                    ok = __all_sync(kAll, mbar_wait(smem_u32(&aux->full[seq % kTilesInFlight]),
                                                    (seq / kTilesInFlight) & 1u, abort_flag)) && ok;
                }
                tc_fence_after();
                uint32_t issue = (ok && do_pv) ? elected : 0u;
                issue_pv_rolled(s, issue, i > 0 ? 1u : 0u);
                umma_commit_if(i == n_it[s] - 1 ? issue : 0u, smem_u32(&aux->o_done[s]));   // only the segment end waits for it
                umma_commit_if(last_reader ? issue : 0u, smem_u32(&aux->empty[v_slot[s]]));
                if (do_pv) advance(v_slot[s]);
                if (i >= 0 && do_qk) { wait_next_k(s, i); tc_fence_after(); }
                issue = (ok && do_qk) ? elected : 0u;
                issue_qk_rolled(s, issue);
                umma_commit_if(issue, smem_u32(&aux->s_full[s]));
                umma_commit_if(last_reader ? issue : 0u, smem_u32(&aux->empty[k_slot[s]]));
                if (do_qk) advance(k_slot[s]);
            }
        };
#pragma unroll 1
        for (int i = -1; i < n_it[0]; ++i) {
            if (i < 0 || i >= n_it[1] - 1) { general(i); continue; }
            // Steady state: both streams have both products.  (Releasing the ring slots from a softmax thread instead -
            // a score tile's arrival covers every product issued before it - would spare this warp two commits of 60 to
            // 100 clocks per tile, but the slots then come back late and the ring runs dry: 15 to 35 % slower.)
            auto steady = [&]() {
                const uint32_t issue = ok ? elected : 0u;
#pragma unroll
                for (int s = 0; s < 2; ++s) {
                    asm volatile("bar.sync %0, 160;" ::"r"(4 + s) : "memory");
                    tc_fence_after();
                    issue_pv(s, issue, i > 0 ? 1u : 0u);
                    if (!shared || s == 1) umma_commit_if(issue, smem_u32(&aux->empty[v_slot[s]]));
                    advance(v_slot[s]);
                    wait_next_k(s, i);                                      // the next K tile has landed
                    issue_qk(s, ok ? issue : 0u);
                    umma_commit_if(issue, smem_u32(&aux->s_full[s]));
                    if (!shared || s == 1) umma_commit_if(issue, smem_u32(&aux->empty[k_slot[s]]));
                    advance(k_slot[s]);
                }
            };
            // (The backward branch over this long unrolled body stalls the warp for some 400 clocks - the loop head has
            // left the instruction caches by the time it is taken.  Two tiles per trip halve the count of branches but
            // double the text; measured, neither form wins.)
            steady();
        }
        item_base += 2u * (uint32_t)T;
        ++seg_no;
    }
}

// ------------------------------------------------------------------------------------------ softmax warpgroups
__device__ __forceinline__ void named_barrier(int id, int count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

__device__ __forceinline__ float max3(float a, float b, float c) { return fmaxf(fmaxf(a, b), c); }

// Writes a warp's 32 rows x 32 columns (lane = row, v = its 32 fp32 values) to global memory through a
// per-warp staging area in shared memory, so that every store instruction covers whole 64- or 128-byte
// row segments instead of 32 scattered 16-byte pieces.  `out_row` / `row_ok` are the lane's own row;
// the other rows' values come by shuffle.  kFinal: bf16 into `out`; else fp32 into the partial slot,
// whose rows are consecutive (part_row0 = row of lane 0).
constexpr int kStageStride = 36;                     // floats per staged row: 16-byte aligned, conflict-free
constexpr int kStageBytesPerWarp = 32 * kStageStride * 4;
// Two floats to two 16-bit values of the cache's element type (x in the low half), round to nearest even.
template <bool kF16>
__device__ __forceinline__ uint32_t pack2_16bit(float x, float y) {
    if (kF16) { __half2 h = __floats2half2_rn(x, y); return *reinterpret_cast<uint32_t*>(&h); }
    __nv_bfloat162 b = __floats2bfloat162_rn(x, y);
    return *reinterpret_cast<uint32_t*>(&b);
}

template <bool kFinal, bool kF16>
__device__ __forceinline__ void store_rows32(const AttnParams& p, float* stage, long long out_row, bool row_ok,
                                             long long part_row0, int col, const float (&v)[32]) {
    const int lane = threadIdx.x & 31;
    __syncwarp();
#pragma unroll
    for (int j = 0; j < 8; ++j)
        *reinterpret_cast<float4*>(stage + lane * kStageStride + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
    __syncwarp();
    // (rolled: this code runs a few times per launch, with cold instruction caches, where its length counts)
    if (kFinal) {
#pragma unroll 1
        for (int k = 0; k < 4; ++k) {                 // 8 rows x 64 bytes per instruction
            const int row = 8 * k + (lane >> 2), piece = lane & 3;
            const long long orow = __shfl_sync(0xffffffffu, out_row, row);
            const bool ok = __shfl_sync(0xffffffffu, row_ok ? 1 : 0, row) != 0;
            const float4 a = *reinterpret_cast<const float4*>(stage + row * kStageStride + piece * 8);
            const float4 b2 = *reinterpret_cast<const float4*>(stage + row * kStageStride + piece * 8 + 4);
            uint4 u;
            u.x = pack2_16bit<kF16>(a.x, a.y); u.y = pack2_16bit<kF16>(a.z, a.w);
            u.z = pack2_16bit<kF16>(b2.x, b2.y); u.w = pack2_16bit<kF16>(b2.z, b2.w);
            if (ok) *reinterpret_cast<uint4*>(p.out + orow * kHeadDim + col + piece * 8) = u;
        }
    } else {
#pragma unroll 2
        for (int k = 0; k < 8; ++k) {                 // 4 rows x 128 bytes per instruction
            const int row = 4 * k + (lane >> 3), piece = lane & 7;
            const bool ok = __shfl_sync(0xffffffffu, row_ok ? 1 : 0, row) != 0;
            const float4 a = *reinterpret_cast<const float4*>(stage + row * kStageStride + piece * 4);
            if (ok) *reinterpret_cast<float4*>(p.part_o + (part_row0 + row) * kHeadDim + col + piece * 4) = a;
        }
    }
}

template <bool kWide, bool kF16>
__device__ __forceinline__ void softmax_loop(const AttnParams& p, Aux* aux, unsigned char* smem, uint32_t tmem, Walker w,
                                             const int s /*stream*/) {
    const int wtid = threadIdx.x - 128 - s * 128;          // 0..127 inside the warpgroup
    const int row_local = wtid;                             // TMEM lane = (warp % 4) * 32 + lane
    volatile int* abort_flag = &aux->abort_flag;
    const uint32_t lane_sel = (uint32_t)(((threadIdx.x >> 5) & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_sel + s * 128;
    const float scale2 = p.sm_scale * 1.4426950408889634f;   // > 0 (checked on the host)
    const int G = p.group;
    uint32_t it = 0, seg_no = 0, od_phase = 0;   // od_phase: segments of this stream that issued a product
    uint32_t tile_base = 0;                      // key tiles of the CTA's earlier segments (the ring counts them through)
    Segment g;

    while (w.template next<kWide>(p, g)) {
        // ---- Q rows (16-byte asynchronous copies, rows beyond M zero-filled) and, in stream 0's warpgroup, the
        // ancestor masks; every global read of the segment start is in flight at the same time
        int parent_i = -1;
        if (s == 0 && wtid < g.n) parent_i = p.tree_parent[g.node_base + wtid];
        if (seg_no > 0) named_barrier(1, 256);   // the other warpgroup may still be reading its staging area in the Q blocks
        {
            // shared: this warpgroup loads its own 128-row block; split: rows [64 s, 64 s + 64) of block 0
            const int blk = g.shared ? s : 0;
            const int r_first = (g.shared ? 0 : 64 * s) + (wtid >> 4);
            const int r_count = g.shared ? 16 : 8;                 // rows per thread, 8 apart
            const int c = wtid & 15;                               // 16-byte chunk of the row
            const uint32_t qs = smem_u32(smem) + blk * kQBytes + (c >> 3) * 16384;
#pragma unroll 2
            for (int j = 0; j < r_count; ++j) {
                const int r = r_first + 8 * j;
                const unsigned rr = (unsigned)(blk * 128 + r);
                const bool valid = rr < (unsigned)g.M;
                const unsigned node = rr / (unsigned)G, hg = rr - node * (unsigned)G;
                const __nv_bfloat16* src =
                    valid ? p.q + ((long long)(g.node_base + node) * p.num_q_heads + g.h * G + hg) * kHeadDim + c * 8 : p.q;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(qs + r * 128 + (((c & 7) ^ (r & 7)) << 4)),
                             "l"(src), "r"(valid ? 16 : 0) : "memory");
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        if (s == 0) {
            if (wtid == 0) aux->seg_bad_tree = 0;
            named_barrier(2, 128);
            if (wtid < g.n) {
                const bool bad = (wtid == 0 && parent_i != -1) || (wtid > 0 && (parent_i < 0 || parent_i >= wtid));
                if (bad) {
                    atomicExch(&aux->seg_bad_tree, 1);
                    report(p.status, kErrBadTree);
                    p.seq_bad[g.b] = p.epoch;
                }
                aux->parent[wtid] = bad ? (short)-1 : (short)parent_i;
            }
            named_barrier(2, 128);
            if (wtid < g.n) {
                unsigned long long m = 0;
                if (!aux->seg_bad_tree)
                    for (int j = wtid, guard = 0; j >= 0 && guard < kMaxNodes; j = aux->parent[j], ++guard) m |= 1ull << j;
                aux->anc[wtid] = m;
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        fence_proxy_async_smem();
        named_barrier(1, 256);                 // masks and the tree verdict are visible to both warpgroups
        mbar_arrive(smem_u32(&aux->q_full));

        const int rr = (g.shared ? s * 128 : 0) + row_local;       // packed row of this thread
        const unsigned long long anc_row = rr < g.M ? aux->anc[rr / G] : 0ull;
        const bool bad_tree = aux->seg_bad_tree != 0;
        const int n_it = g.iters(s);
        float m = -INFINITY, l = 0.f, lx = 0.f;   // l: sum of the bf16 weights (normaliser); lx: exact sum (LSE)

        for (int i = 0; i < n_it; ++i) {
            const int t = g.tile(s, i);
            mbar_wait(smem_u32(&aux->s_full[s]), it & 1u, abort_flag);
            tc_fence_after();
            if ((t + 1) * kTileKeys > g.L) {
                // The tile reaches drafted positions (or the end of the sequence): at most two tiles per unit.
                // Visibility of its 128 keys for this row: prefix keys all, drafted key j iff ancestor-or-self.
                // The mask is applied to S in tensor memory, 32 columns at a time, before the common path reads it.
                const int j0 = t * kTileKeys - g.L;
                unsigned long long lo, hi;
                if (j0 >= 0) {
                    lo = j0 < 64 ? anc_row >> j0 : 0ull;
                    hi = 0ull;
                } else {
                    const int k = -j0;   // 1..127 prefix keys at the front of the tile
                    if (k >= 64) { lo = ~0ull; hi = (k == 64 ? 0ull : (~0ull >> (128 - k))) | (anc_row << (k - 64)); }
                    else { lo = (~0ull >> (64 - k)) | (anc_row << k); hi = anc_row >> (64 - k); }
                }
#pragma unroll 1
                for (int c4 = 0; c4 < 4; ++c4) {
                    const uint32_t bits = (uint32_t)((c4 < 2 ? lo : hi) >> ((c4 & 1) * 32));
                    uint32_t r[32];
                    tmem_ld32(tS + c4 * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (!((bits >> j) & 1u)) r[j] = 0xff800000u;   // -inf
                    tmem_st32(tS + c4 * 32, r);
                }
                tmem_wait_st();
                // Slots of the sequence's last page beyond L + n may hold anything, NaN and Inf included.  Their scores
                // were just overwritten (weight exactly 0), but 0 * NaN would still reach O through P V: zero those
                // V rows in the ring slot (pages wholly past the end were zero-filled by the copy itself).  The
                // tile's arrival barrier covers V as well as K, so the rows have landed; the stores are ordered
                // before the product by the proxy fence here and the hand-off of P below.  Both warpgroups of a
                // 256-row unit do it (zeros over zeros); the slot is not released before both products are done.
                const int kv_valid = g.L + g.n - t * kTileKeys;            // >= 1 valid keys in this tile
                if (kv_valid < kTileKeys) {
                    const int kv_end = min(kTileKeys, ((kv_valid + p.page_size - 1) >> p.page_shift) << p.page_shift);
                    const uint32_t seq = tile_base + (uint32_t)(g.shared ? i : 2 * i + s);
                    unsigned char* vslot = smem + kRingOff + ((2u * seq + 1u) % kSlots) * kSlotBytes;
#pragma unroll 1
                    for (int k = kv_valid + (wtid >> 4); k < kv_end; k += 8)   // 16 threads x 16 bytes per 256-byte row
                        *reinterpret_cast<uint4*>(vslot + (k >> 3) * 2048 + ((wtid >> 3) & 1) * 1024 + (k & 7) * 128 +
                                                  (wtid & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
                    fence_proxy_async_smem();
                }
            }
            // Fast path (every tile but a segment's first, as long as the running maximum holds): the weights are
            // computed against the running maximum m straight away, 32 columns at a time while the next 32 are on
            // their way from tensor memory, with no pass for the tile's own maximum.  A softmax job is what the products
            // of its stream wait for, and every instruction of it also competes with the MMA warp for the issue slots
            // of their SM sub-partition.  If some row's weights add up to more than 2^8 (some score may then exceed m
            // by more than the lazy threshold; rare after the first tiles), nothing has been stored yet and the tile
            // is redone the long way.
            bool done = false, force = false;
            if (i > 0 && !__any_sync(0xffffffffu, m == -INFINITY)) {
                const uint64_t scale2_x2 = pack_f32x2(scale2, scale2), neg_m_x2 = pack_f32x2(-m, -m);
                uint64_t ex_a = 0ull, ex_b = 0ull, rs_a = 0ull, rs_b = 0ull;
                uint32_t pk[64];
                uint32_t buf_a[32], buf_b[32];
                tmem_ld32(tS, buf_a);
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint32_t (&cur)[32] = (c4 & 1) ? buf_b : buf_a;
                    uint32_t (&nxt)[32] = (c4 & 1) ? buf_a : buf_b;
                    tmem_wait_ld();
                    if (c4 < 3) tmem_ld32(tS + (c4 + 1) * 32, nxt);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        float x0, x1;
                        const uint64_t xx = fma_f32x2(pack_f32x2(__uint_as_float(cur[2 * j]), __uint_as_float(cur[2 * j + 1])),
                                                      scale2_x2, neg_m_x2);
                        unpack_f32x2(xx, x0, x1);
                        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                        const uint32_t u = pack2_16bit<kF16>(p0, p1);
                        pk[c4 * 16 + j] = u;
                        const uint64_t pe = pack_f32x2(p0, p1);
                        uint64_t pr;      // the two weights as the tensor core will read them
                        if (kF16) {
                            const float2 r = __half22float2(*reinterpret_cast<const __half2*>(&u));
                            pr = pack_f32x2(r.x, r.y);
                        } else {
                            pr = pack_f32x2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
                        }
                        if (j & 1) { ex_b = add_f32x2(ex_b, pe); rs_b = add_f32x2(rs_b, pr); }
                        else { ex_a = add_f32x2(ex_a, pe); rs_a = add_f32x2(rs_a, pr); }
                    }
                }
                float a0, a1, b0, b1;
                unpack_f32x2(add_f32x2(rs_a, rs_b), a0, a1);
                unpack_f32x2(add_f32x2(ex_a, ex_b), b0, b1);
                // no weight can exceed the tile's sum: a sum of at most 2^8 means that no score is more than the lazy
                // threshold above m (a larger sum sends the tile the long way, which then moves m up)
                force = (b0 + b1) > 256.f;
                if (!__any_sync(0xffffffffu, force)) {
                    tmem_st32(tS, reinterpret_cast<uint32_t(&)[32]>(pk[0]));
                    tmem_st32(tS + 32, reinterpret_cast<uint32_t(&)[32]>(pk[32]));
                    l += a0 + a1;
                    lx += b0 + b1;
                    done = true;
                }
            }
            if (!done) {
                // The long way: the tile's maximum first, then the weights; twice over tensor memory and rolled, because
                // it runs on a segment's first tile and after a jump of the maximum only - its length in the kernel's
                // text costs every launch more than its speed gains.
                float mx = -INFINITY;
#pragma unroll 1
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint32_t r[32];
                    tmem_ld32(tS + c4 * 32, r);
                    tmem_wait_ld();
                    float a = max3(__uint_as_float(r[0]), __uint_as_float(r[1]), __uint_as_float(r[2])), b = __uint_as_float(r[3]);
#pragma unroll
                    for (int j = 4; j + 3 < 32; j += 4) {
                        a = max3(a, __uint_as_float(r[j]), __uint_as_float(r[j + 1]));
                        b = max3(b, __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
                    }
                    mx = max3(mx, a, b);
                }
                const float m_new = fmaxf(m, mx * scale2);
                // (false when both are -inf: NaN compares false)  A tile sent here by the fast path's sum moves m up at once.
                const bool need = force ? m_new > m : (m_new - m) > kLazyRescale;
                if (__any_sync(0xffffffffu, need)) {
                    const float alpha = (m_new == -INFINITY) ? 1.f : fast_exp2(m - m_new);
                    if (i > 0) {
                        // S of this tile is here, and its product was issued after O += P V of the tile before: the
                        // commit that announced S covers that product too, so O may be touched now
                        tc_fence_after();
                        const uint32_t tO = tmem + lane_sel + 256 + s * 128;
#pragma unroll 1
                        for (int c4 = 0; c4 < 4; ++c4) {
                            uint32_t o[32];
                            tmem_ld32(tO + c4 * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
                            tmem_st32(tO + c4 * 32, o);
                        }
                        tmem_wait_st();
                        l *= alpha;
                        lx *= alpha;
                    }
                    m = m_new;
                }
                const float neg_m = (m == -INFINITY) ? 0.f : -m;
                const uint64_t scale2_x2 = pack_f32x2(scale2, scale2), neg_m_x2 = pack_f32x2(neg_m, neg_m);
                // two packed accumulators each for the exact sum (LSE) and for the sum of the rounded weights: the
                // normaliser takes the very numbers P V multiplies by, so that out = sum(p v) / sum(p) stays a true
                // weighted mean (exact when one key dominates)
                uint64_t ex_a = 0ull, ex_b = 0ull, rs_a = 0ull, rs_b = 0ull;
#pragma unroll 1
                for (int hf = 0; hf < 2; ++hf) {
                    // keys [64 hf, 64 hf + 64) lie in columns the weights written so far (columns below 32 hf) do not reach
                    uint32_t sv[64], pk[32];
                    tmem_ld64(tS + hf * 64, sv);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        float x0, x1;
                        const uint64_t xx = fma_f32x2(pack_f32x2(__uint_as_float(sv[2 * j]), __uint_as_float(sv[2 * j + 1])), scale2_x2, neg_m_x2);
                        unpack_f32x2(xx, x0, x1);
                        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                        const uint32_t u = pack2_16bit<kF16>(p0, p1);
                        pk[j] = u;
                        const uint64_t pe = pack_f32x2(p0, p1);
                        uint64_t pr;      // the two weights as the tensor core will read them
                        if (kF16) {
                            const float2 r = __half22float2(*reinterpret_cast<const __half2*>(&u));
                            pr = pack_f32x2(r.x, r.y);
                        } else {
                            pr = pack_f32x2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
                        }
                        if (j & 1) { ex_b = add_f32x2(ex_b, pe); rs_b = add_f32x2(rs_b, pr); }
                        else { ex_a = add_f32x2(ex_a, pe); rs_a = add_f32x2(rs_a, pr); }
                    }
                    tmem_st32(tS + hf * 32, pk);
                }
                {
                    float a0, a1, b0, b1;
                    unpack_f32x2(add_f32x2(rs_a, rs_b), a0, a1);
                    unpack_f32x2(add_f32x2(ex_a, ex_b), b0, b1);
                    l += a0 + a1;
                    lx += b0 + b1;
                }
            }
            tmem_wait_st();
            tc_fence_before();
            // Hand-off of P: hardware barrier 4 + s, 160 threads (this warpgroup + the MMA warp).  Executed once per
            // key tile of this stream - n_it times per segment, the count of the MMA warp's bar.sync on it - on every
            // path: nothing above leaves the loop body early, and a wait that gave up only changed what was computed.
            asm volatile("bar.arrive %0, 160;" ::"r"(4 + s) : "memory");
            // In a unit of more than 128 rows the MMA warp polls no mbarrier between O += P V of this tile and
            // S = Q K^T of the next one: the first warp of the warpgroup looks at that tile's arrival barrier for it
            // (after P is announced, so that nothing this tile holds is released any later) and passes the news on
            // through hardware barrier 6 (stream 0's warpgroup does; the tile is the same for both streams).  A wait
            // that gives up raises the abort flag; the arrival happens all the same.
            if (g.shared && s == 0 && wtid < 32 && i + 1 < n_it) {
                const uint32_t seq = tile_base + (uint32_t)(i + 1);
                mbar_wait(smem_u32(&aux->full[seq % kTilesInFlight]), (seq / kTilesInFlight) & 1u, abort_flag);
                // hardware barrier 6, 64 threads (this warp + the MMA warp): once per tile but the segment's last,
                // T - 1 times, matching the MMA warp's bar.sync 6 before S of tiles 1 .. T - 1; unconditional
                asm volatile("bar.arrive 6, 64;" ::: "memory");
            }
            ++it;
        }

        // ---- segment end: every product of this stream has completed
        if (n_it > 0) { mbar_wait(smem_u32(&aux->o_done[s]), od_phase & 1u, abort_flag); ++od_phase; }
        tc_fence_after();
        // split mode: the streams exchange (m, l, lx) through the second Q block, which only the shared mode uses
        float (*ml)[128][3] = reinterpret_cast<float (*)[128][3]>(smem + kQBytes);
        if (!g.shared) { ml[s][row_local][0] = m; ml[s][row_local][1] = l; ml[s][row_local][2] = lx; }
        named_barrier(1, 256);                 // both streams done: all MMAs of the segment have completed
        const bool write_ok = !bad_tree && !*abort_flag && *reinterpret_cast<volatile int32_t*>(p.seq_bad + g.b) != p.epoch;
        // only the first and the last unit of a CTA's piece can be cut: two partial slots per CTA
        const long long part_row = (2ll * blockIdx.x + (seg_no > 0 ? 1 : 0)) * p.rows_per_slot + rr;
        const long long out_row = rr < g.M ? (long long)(g.node_base + rr / G) * p.num_q_heads + g.h * G + rr % G : 0;
        const bool row_ok = write_ok && rr < g.M;
        const bool whole = g.whole();
        // staging for coalesced stores: the Q blocks are idle now (every MMA of the segment is done); stream 1's
        // area starts after the (m, l, lx) exchange
        float* stage = reinterpret_cast<float*>(smem + s * (kQBytes + 4096) + ((threadIdx.x >> 5) & 3) * kStageBytesPerWarp);
        const long long part_row0 = part_row - (threadIdx.x & 31);
        // One loop writes both modes.  shared: this warpgroup's own rows, all 128 columns of its O, weight 1 / l.
        // split: the two streams hold the same rows over disjoint key tiles; they are merged by their maxima and
        // sums, and this warpgroup writes columns [64 s, 64 s + 64) of the merged rows.
        float wa, wb = 0.f, lse;
        uint32_t tOa = tmem + lane_sel + 256 + s * 128, tOb = tmem + lane_sel + 384;
        bool use_b = false, write_lse = true;
        int c_first = 0, c_count = 4;
        if (g.shared) {
            wa = l > 0.f ? 1.f / l : 0.f;
            lse = lx > 0.f ? (m + __log2f(lx)) * 0.6931471805599453f : -INFINITY;
        } else {
            const float m0 = ml[0][row_local][0], l0 = ml[0][row_local][1], x0 = ml[0][row_local][2];
            use_b = g.iters(1) > 0;
            const float m1 = use_b ? ml[1][row_local][0] : -INFINITY, l1 = use_b ? ml[1][row_local][1] : 0.f;
            const float x1 = use_b ? ml[1][row_local][2] : 0.f;
            const float mm = fmaxf(m0, m1);
            const float a0 = (m0 == -INFINITY) ? 0.f : fast_exp2(m0 - mm);
            const float a1 = (m1 == -INFINITY) ? 0.f : fast_exp2(m1 - mm);
            const float lt = a0 * l0 + a1 * l1, xt = a0 * x0 + a1 * x1;
            const float inv = lt > 0.f ? 1.f / lt : 0.f;
            wa = a0 * inv; wb = a1 * inv;
            lse = xt > 0.f ? (mm + __log2f(xt)) * 0.6931471805599453f : -INFINITY;
            tOa = tmem + lane_sel + 256;
            write_lse = s == 0;
            c_first = 2 * s; c_count = 2;
        }
#pragma unroll 1
        for (int c4 = c_first; c4 < c_first + c_count; ++c4) {
            uint32_t oa[32], ob[32];
            tmem_ld32(tOa + c4 * 32, oa);
            if (use_b) tmem_ld32(tOb + c4 * 32, ob);
            tmem_wait_ld();
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                v[j] = __uint_as_float(oa[j]) * wa;           // rows that saw no key have O = 0 and weight 0
                if (use_b) v[j] = fmaf(__uint_as_float(ob[j]), wb, v[j]);
            }
            if (whole) store_rows32<true, kF16>(p, stage, out_row, row_ok, part_row0, c4 * 32, v);
            else store_rows32<false, kF16>(p, stage, out_row, row_ok, part_row0, c4 * 32, v);
        }
        if (row_ok && write_lse) {
            if (whole) { if (p.lse) p.lse[out_row] = lse; }
            else p.part_lse[part_row] = lse;
        }
        tc_fence_before();
        tile_base += (uint32_t)(g.tile1 - g.tile0);
        ++seg_no;
    }
}

// ------------------------------------------------------------------------------------------ kernel
// kManySeqs: more than 32 sequences (the block-wide schedule); kWide: some unit may have more than 128 rows.
// Separate instances, so that a launch carries only the code of its own case: the text of the paths a launch never takes
// still costs it time (3 us of 39 on a 32K-context, 32-node step when the block-wide schedule was compiled in).
// kFused: the verify step's logits scan rides along.  Warps 2 and 3 have no part in the attention; they take the
// (row, vocabulary chunk) items of the arg-max scan in turn, 2 x gridDim.x warps in all, and leave one key per item
// for the acceptance walk, which the merge kernel runs after this grid (`ap` is not looked at otherwise).
// kF16: q, the caches and out are fp16 instead of bf16 (the weights P are then rounded to fp16 as well).
template <bool kManySeqs, bool kWide, bool kFused, bool kF16>
__global__ void __launch_bounds__(kThreads, 1)
verify_attn_umma_kernel(const AttnParams p, const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap,
                        const AcceptParams ap) {
    extern __shared__ __align__(1024) unsigned char smem[];
    Aux* aux = reinterpret_cast<Aux*>(smem + kAuxOff);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = smem_u32(smem);
    if (smem_base & 1023u) {                       // operand tiles must sit on swizzle-atom boundaries
        if (tid == 0) report(p.status, kErrTimeout);
        return;
    }
    if (tid == 0) {
        for (int i = 0; i < kSlots; ++i) mbar_init(smem_u32(&aux->empty[i]), 1);
        for (int i = 0; i < kTilesInFlight; ++i) mbar_init(smem_u32(&aux->full[i]), 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&aux->s_full[s]), 1);
            mbar_init(smem_u32(&aux->o_done[s]), 1);
        }
        mbar_init(smem_u32(&aux->q_full), 256);
        aux->abort_flag = 0;
        aux->seg_bad_tree = 0;
        aux->sched_b0 = 0; aux->sched_tile_begin = 0; aux->sched_unit_begin = 0;
        fence_barrier_init();
        tma_prefetch_desc(&kmap);
        tma_prefetch_desc(&vmap);
    }
    if (warp == 0) { tmem_alloc(smem_u32(&aux->tmem_base), kTmemCols); tmem_relinquish(); }
    // launched as a programmatic dependent itself: everything above touched no input; from here on the kernel
    // before this one in the stream has completed (a no-op in an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // The combine kernel is launched as a programmatic dependent and may queue up behind this grid's CTAs from here
    // on.  It reads the call's inputs (lengths, offsets) before its own wait: triggering only after this grid's wait
    // keeps those reads ordered after whatever kernel wrote them earlier in the stream.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    Walker w;
    if (!kManySeqs) build_walk_small(p, w);        // its global loads overlap the set-up above
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = aux->tmem_base;
    if (kManySeqs) build_walk(p, aux, w);

    // registers move from the warpgroup of the producer / MMA warps to the two softmax warpgroups,
    // whose threads each hold a 128-column row of S: 128 x 72 + 256 x 216 = 384 x 168, the registers the CTA was launched with
    uint32_t items = 0;
    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
        if (warp == 0) producer_loop<kWide>(p, &kmap, &vmap, aux, smem_base + kRingOff, w, items);
        else if (warp == 1) mma_loop<kWide, kF16>(p, aux, smem_base, tmem, w);
        else if (kFused) {
            const long long items = (long long)ap.total_nodes * ap.chunks;
            for (long long it = 2ll * blockIdx.x + (warp - 2); it < items; it += 2ll * gridDim.x)
                argmax_scan_chunk_warp<false>(ap, (int)(it / ap.chunks), (int)(it % ap.chunks));
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        softmax_loop<kWide, kF16>(p, aux, smem, tmem, w, warp >= 8 ? 1 : 0);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        if (aux->abort_flag) {
            // give the copies still in flight a bounded time to land before the CTA's shared memory is released
            const uint32_t tiles_issued = (items + 1u) >> 1;
            const uint32_t first = tiles_issued > (uint32_t)kTilesInFlight ? tiles_issued - kTilesInFlight : 0u;
            for (uint32_t it = first; it < tiles_issued; ++it) {
                const uint32_t bar = smem_u32(&aux->full[it % kTilesInFlight]), ph = (it / kTilesInFlight) & 1u;
                for (int polls = 0; polls < (1 << 20) && !mbar_try_wait(bar, ph); ++polls) {}
            }
            if (lane == 0) report(p.status, kErrTimeout);
        }
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

}  // namespace umma_path
}  // namespace owl
