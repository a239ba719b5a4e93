// Shared device/host helpers of libowlverify: work partition of the split-KV pass,
// status reporting, small PTX wrappers.  sm_100a only.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace owl {

constexpr int kHeadDim = 128;
constexpr int kMaxNodes = 64;     // drafted nodes per sequence (the paper's trees have 60)
constexpr int kMaxBatch = 1024;   // sequences per call (schedule prefix sums live in shared memory)
constexpr int kMaxRows = 256;     // packed rows (query heads of a KV group x nodes) per (sequence, KV head)

// Device-detected status codes: same values as owl_status in owlverify.h.
constexpr int kErrBadTree = -4;
constexpr int kErrBadPage = -5;
constexpr int kErrTimeout = -6;

struct SchedHeader;

// Problem description handed to every kernel of the attention path.
struct AttnParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_cache;
    const __nv_bfloat16* v_cache;
    const int32_t* block_table;
    const int32_t* ctx_lens;
    const int32_t* node_offsets;  // may be null: uniform nodes_uniform per sequence
    const int32_t* tree_parent;
    __nv_bfloat16* out;
    float* lse;                   // may be null
    float* part_o;                // [slots, rows_per_slot, D] fp32, normalised partial outputs
    float* part_lse;              // [slots, rows_per_slot] fp32, natural-log partial LSE (-inf if empty)
    int32_t* status;              // device status word (0 = ok, first error wins)
    int32_t* seq_bad;             // [B] epoch of the call in which the sequence was found malformed
    long long* sched_seq_begin;   // [B + 1] first flat tile of every sequence (written by CTA 0 of the pass)
    SchedHeader* sched_header;
    int32_t epoch;
    int32_t batch, total_nodes, nodes_uniform, max_nodes;
    int32_t num_q_heads, num_kv_heads, group;  // group = Hq / Hkv
    int32_t page_size, page_shift, max_pages_per_seq, num_pages;
    int32_t rows_per_slot;        // row stride of one partial slot
    int32_t num_ctas;             // CTAs of the split-KV pass (the flat tile range is cut into this many pieces)
    int32_t combine_row_ctas;     // CTAs of the merge kernel that take output rows (persistent, eight warps each)
    int32_t f16;                  // q / caches / out are fp16 instead of bf16 (same size; typed as bf16 pointers here)
    float sm_scale;
};

// 2^x by the special-function unit (ex2.approx, denormals flushed); ex2(-inf) = 0.
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void report(int32_t* status, int code) { atomicCAS(status, 0, code); }

// ---------------------------------------------------------------------------------------------
// Flat partition of the split-KV pass.
//
// A unit is (sequence b, KV head h) with all its G * n_b packed rows; it owns
// tiles_b = ceil((L_b + n_b) / TileKeys) key tiles.  Units are laid out sequence-major, then head;
// all their tiles form one flat range [0, total) which is cut into num_ctas contiguous pieces.  A
// CTA's piece may start and end inside a unit; only its first and its last unit can be cut, so a
// CTA stores at most two partials (o, lse): slot 2c for the unit its piece starts in, 2c + 1 for a later one.
// ---------------------------------------------------------------------------------------------
// Cut of the flat tile range [0, total) into `ctas` pieces, one per CTA.
//   flat:    contiguous, nearly equal pieces; a piece may start and end inside a unit.
//   aligned: only when every unit has the same number of tiles (`unit_tiles`) and there are at least as
//            many CTAs as units: unit u is cut into base + (u < urem) nearly equal pieces, so no piece
//            crosses a unit boundary.  Chosen when its largest piece is smaller than the flat piece plus
//            what a unit boundary costs a CTA (pipeline drain, epilogue, new Q), counted in tiles.
constexpr int kBoundaryPenaltyTiles = 5;
struct Partition {
    long long total, q;
    int rem, ctas;
    int unit_tiles, base, urem;   // aligned mode iff unit_tiles > 0
    // (Every CTA runs this once, on its critical path and with cold instruction caches, where each instruction costs
    // tens of nanoseconds: one 32-bit division where the numbers allow it instead of 64-bit ones.)
    __device__ __host__ void init(long long total_, int ctas_) {
        total = total_; ctas = ctas_;
        if (total_ >= 0 && total_ <= 0x7fffffffll) {
            const unsigned qq = (unsigned)total_ / (unsigned)ctas_;
            q = qq; rem = (int)((unsigned)total_ - qq * (unsigned)ctas_);
        } else {
            q = total_ / ctas_; rem = (int)(total_ % ctas_);
        }
        unit_tiles = 0; base = 0; urem = 0;
    }
    __device__ __host__ void init(long long total_, int ctas_, int units, int uniform_tiles) {
        init(total_, ctas_);
        if (uniform_tiles > 0 && units > 1 && units <= ctas_) {
            const int b = ctas_ / units;
            const long long cost_aligned = (uniform_tiles + b - 1) / b;
            const long long cost_flat = q + (rem ? 1 : 0) + kBoundaryPenaltyTiles;   // ceil(total / ctas) + penalty
            if (cost_aligned < cost_flat) { unit_tiles = uniform_tiles; base = b; urem = ctas_ - b * units; }
        }
    }
    // [begin(c), begin(c + 1)) with one set of divisions (the pieces of a unit tile it exactly, so a piece's end is
    // its begin plus its length in either mode)
    __device__ __host__ void range(int c, long long& t_begin, long long& t_end) const {
        if (unit_tiles == 0) {
            t_begin = (long long)c * q + (c < rem ? c : rem);
            t_end = t_begin + q + (c < rem ? 1 : 0);
            return;
        }
        const int big = urem * (base + 1);
        int u, k, cu;
        if (c < big) { u = c / (base + 1); k = c - u * (base + 1); cu = base + 1; }
        else { u = urem + (c - big) / base; k = (c - big) - (u - urem) * base; cu = base; }
        const int qq = unit_tiles / cu, rr = unit_tiles - qq * cu;
        t_begin = (long long)u * unit_tiles + (long long)k * qq + (k < rr ? k : rr);
        t_end = t_begin + qq + (k < rr ? 1 : 0);
    }
    __device__ __host__ long long begin(int c) const {
        if (unit_tiles == 0) return (long long)c * q + (c < rem ? c : rem);
        const int big = urem * (base + 1);
        int u, k, cu;
        if (c < big) { u = c / (base + 1); k = c - u * (base + 1); cu = base + 1; }
        else { u = urem + (c - big) / base; k = (c - big) - (u - urem) * base; cu = base; }
        const int qq = unit_tiles / cu, rr = unit_tiles % cu;
        return (long long)u * unit_tiles + (long long)k * qq + (k < rr ? k : rr);
    }
    __device__ __host__ int owner(long long t) const {
        if (unit_tiles == 0) {
            long long big = (long long)rem * (q + 1);
            if (total <= 0x7fffffffll) {      // the usual case: 32-bit divisions
                const unsigned tt = (unsigned)t, qq = (unsigned)q, bb = (unsigned)big;
                return tt < bb ? (int)(tt / (qq + 1u)) : rem + (int)((tt - bb) / qq);
            }
            return t < big ? (int)(t / (q + 1)) : rem + (int)((t - big) / q);
        }
        const int u = total <= 0x7fffffffll ? (int)((unsigned)t / (unsigned)unit_tiles) : (int)(t / unit_tiles);
        const int local = (int)(t - (long long)u * unit_tiles);
        const int cu = base + (u < urem ? 1 : 0), c0 = u * base + (u < urem ? u : urem);
        const int qq = unit_tiles / cu, rr = unit_tiles % cu, bigl = rr * (qq + 1);
        return c0 + (local < bigl ? local / (qq + 1) : rr + (local - bigl) / qq);
    }
};

// What the split-KV pass leaves for the combine kernel: totals and the choice of partition.
struct SchedHeader {
    long long total_tiles;
    int uniform_tiles;   // tiles per unit if every schedulable sequence has the same count, else 0
    int units;
};

__device__ __forceinline__ int seq_nodes(const AttnParams& p, int b) {
    return p.node_offsets ? p.node_offsets[b + 1] - p.node_offsets[b] : p.nodes_uniform;
}
__device__ __forceinline__ int seq_node_base(const AttnParams& p, int b) {
    return p.node_offsets ? p.node_offsets[b] : b * p.nodes_uniform;
}

// A sequence is schedulable when its node count and lengths are inside the interface's limits.
__device__ __forceinline__ bool seq_tree_shape_ok(const AttnParams& p, int b, int n) {
    const int base = seq_node_base(p, b);
    return n >= 1 && n <= p.max_nodes && base >= 0 && base + n <= p.total_nodes;
}
__device__ __forceinline__ bool seq_shape_ok(const AttnParams& p, int b, int n, int L) {
    if (!seq_tree_shape_ok(p, b, n) || L < 0) return false;
    long long keys = (long long)L + n;
    return keys <= (long long)p.max_pages_per_seq * p.page_size;
}

// Schedule of a batch of at most 32 sequences, derived by one warp on its own: lane b holds sequence b, prefix sums
// by shuffle, no shared memory.  The split-KV pass (every warp of it) and the merge that follows it call the same
// function on the same inputs, so the merge needs nothing from the pass but its partials.
constexpr int kSchedTileKeys = 128;      // key tile of the split-KV pass
struct WarpSchedule {
    int n, L, node_base, tiles;          // this lane's sequence (tiles = 0 if it is not schedulable)
    bool ok;
    long long my_tiles, excl_t, total;   // flat tiles of this sequence (all KV heads), of the ones before it, of all
    int my_units, excl_u, units;
    int uniform_tiles;                   // tiles per unit if every schedulable sequence has the same count, else 0
};
__device__ __forceinline__ WarpSchedule warp_schedule(const AttnParams& p) {
    const int lane = threadIdx.x & 31;
    WarpSchedule ws;
    ws.n = 0; ws.L = 0; ws.node_base = 0; ws.tiles = 0; ws.ok = false;
    if (lane < p.batch) {
        ws.n = seq_nodes(p, lane);
        ws.L = p.ctx_lens[lane];
        ws.node_base = seq_node_base(p, lane);
        ws.ok = seq_shape_ok(p, lane, ws.n, ws.L);
        ws.tiles = ws.ok ? (ws.L + ws.n + kSchedTileKeys - 1) / kSchedTileKeys : 0;
    }
    ws.my_tiles = (long long)ws.tiles * p.num_kv_heads;
    ws.my_units = ws.ok ? p.num_kv_heads : 0;
    long long inc_t = ws.my_tiles;
    int inc_u = ws.my_units, tmin = ws.ok ? ws.tiles : 0x7fffffff, tmax = ws.ok ? ws.tiles : 0;
    // as many rounds as the batch needs (one sequence: none): this runs once per launch on every CTA's critical
    // path, where an instruction costs tens of nanoseconds.  Lanes >= batch hold zeros / neutral elements.
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        if (o >= p.batch) break;
        const long long vt = __shfl_up_sync(0xffffffffu, inc_t, o);
        const int vu = __shfl_up_sync(0xffffffffu, inc_u, o);
        if (lane >= o) { inc_t += vt; inc_u += vu; }
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {               // after the rounds with o < batch, lane 0 covers [0, batch)
        if (o >= p.batch) break;
        tmin = min(tmin, __shfl_down_sync(0xffffffffu, tmin, o));
        tmax = max(tmax, __shfl_down_sync(0xffffffffu, tmax, o));
    }
    tmin = __shfl_sync(0xffffffffu, tmin, 0);
    tmax = __shfl_sync(0xffffffffu, tmax, 0);
    const int last = p.batch < 32 ? p.batch - 1 : 31;
    ws.total = __shfl_sync(0xffffffffu, inc_t, last);
    ws.units = __shfl_sync(0xffffffffu, inc_u, last);
    ws.uniform_tiles = (ws.units > 0 && tmin == tmax) ? tmin : 0;
    ws.excl_t = inc_t - ws.my_tiles;
    ws.excl_u = inc_u - ws.my_units;
    return ws;
}

}  // namespace owl
