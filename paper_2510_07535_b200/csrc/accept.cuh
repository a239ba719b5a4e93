// Greedy tree acceptance: row arg-max over the vocabulary, then the acceptance walk.
//
// The scan reads fp32 logits with 16-byte loads, one warp per (row, 8192-float vocabulary chunk) item.  Every
// (value, index) candidate is folded into one 64-bit key, high word = the float mapped to an unsigned
// integer that sorts like the float (NaN mapped to -inf, -0 to +0), low word = ~index, so that an unsigned
// max picks the larger value and, among equal values, the lower index.  Per-lane and warp (shuffle) maxima
// give one key per item, stored to part_keys[row][chunk] (no atomics, nothing to initialise).
//
// The warp that stores the last chunk key of a sequence (a per-sequence counter, bumped after a
// __threadfence; nobody waits for anybody) notes the sequence, and its CTA does that sequence's walk in the
// same launch: it reduces the chunk keys to arg-max tokens, evaluates for every node whether all edges on its
// root path match (draft token == parent's arg-max), picks the deepest matching node (lowest index among
// equals) and writes accept_len / accept_path / bonus_token.  Calls alternate between two sets of counters and
// clear the idle one as a whole, so no separate clearing pass is needed.
//
// Inside a verify step with a small scan both halves run as guests of the attention kernels: the scan in warps
// the attention pass does not use (argmax_scan_chunk_warp), the walk in extra CTAs of the merge kernel, after
// the pass has completed; no counters are involved there.
#pragma once

#include "owl_common.cuh"

namespace owl {

constexpr int kArgmaxThreads = 256;
static_assert(kArgmaxThreads >= kMaxNodes, "the walk needs one thread per node");
constexpr int kArgmaxChunk = 8192;  // floats per CTA: 8 x float4 per thread

// 16-byte load of data that is read once: no L1 allocation, first in line for eviction from L2
// (`policy` from createpolicy.fractional.L2::evict_first).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ float4 ld_stream_f4(const float4* ptr, uint64_t policy) {
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr), "l"(policy));
    return v;
}

struct AcceptParams {
    const float* logits;
    const int32_t* draft_tokens;
    const int32_t* node_offsets;
    const int32_t* tree_parent;
    int32_t* accept_len;
    int32_t* accept_path;
    int32_t* bonus_token;
    int32_t* node_argmax;
    int32_t* spec_node;              // optional [B]: the [SPEC] leaf (negative draft token) under the last accepted node
    unsigned long long* part_keys;   // [total_nodes, chunks]
    unsigned int* seq_counter;       // [2, batch]: chunk keys of the sequence stored so far; set epoch & 1 is in use
    uint32_t epoch;                  // call number: the other set is cleared for the next call
    int32_t counter_stride;          // distance between the two sets
    int32_t* status;
    int32_t batch, total_nodes, nodes_uniform, max_nodes, vocab, path_stride, chunks;
};

__device__ __forceinline__ unsigned long long argmax_key(float x, uint32_t idx) {
    if (x != x) x = -INFINITY;   // NaN never wins
    x += 0.0f;                   // -0.0 -> +0.0
    uint32_t u = __float_as_uint(x);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((unsigned long long)u << 32) | (uint32_t)(~idx);
}

// Called by every thread of the CTA (threads >= kMaxNodes only keep the barriers company).
__device__ __forceinline__ void accept_walk_seq(const AcceptParams& p, const int b) {
    const int i = threadIdx.x;
    const int base = p.node_offsets ? p.node_offsets[b] : b * p.nodes_uniform;
    const int n = p.node_offsets ? p.node_offsets[b + 1] - base : p.nodes_uniform;
    __shared__ int s_parent[kMaxNodes], s_am[kMaxNodes], s_tok[kMaxNodes];
    __shared__ int s_bad, s_win, s_leaf;
    if (i == 0) {
        s_bad = (n < 1 || n > p.max_nodes || n > p.path_stride || base < 0 || base + n > p.total_nodes) ? 1 : 0;
        s_win = 0;
        s_leaf = kMaxNodes;
    }
    __syncthreads();
    if (s_bad) { if (i == 0) report(p.status, kErrBadTree); return; }
    if (i < n) {
        const int pi = p.tree_parent[base + i];
        s_parent[i] = pi;
        s_tok[i] = p.draft_tokens[base + i];
        unsigned long long k = 0;
        const unsigned long long* pk = p.part_keys + (long long)(base + i) * p.chunks;
        // independent loads, eight in flight (a dependent one-by-one walk would cost a memory round trip per chunk)
        for (int c0 = 0; c0 < p.chunks; c0 += 8) {
            unsigned long long v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = c0 + j < p.chunks ? __ldcg(pk + c0 + j) : 0ull;
#pragma unroll
            for (int j = 0; j < 8; ++j) k = v[j] > k ? v[j] : k;
        }
        const int am = (int)(~(uint32_t)(k & 0xffffffffull));
        s_am[i] = am;
        if (p.node_argmax) p.node_argmax[base + i] = am;
        if ((i == 0 && pi != -1) || (i > 0 && (pi < 0 || pi >= i))) atomicExch(&s_bad, 1);
    }
    __syncthreads();
    if (s_bad) { if (i == 0) report(p.status, kErrBadTree); return; }

    // ok(i): every edge on the root path of i matches; depth(i): number of edges
    int key = 0;
    if (i < n) {
        bool ok = true;
        int depth = 0;
        for (int c = i; s_parent[c] >= 0 && depth < kMaxNodes; c = s_parent[c], ++depth)
            ok = ok && s_tok[c] >= 0 && s_tok[c] == s_am[s_parent[c]];
        if (ok) key = ((depth + 1) << 8) | (kMaxNodes - 1 - i);   // deeper first, then lower index
    }
    atomicMax(&s_win, key);
    __syncthreads();
    if (p.spec_node) {
        // Section 3.2.2 "Decode Stage": the hidden state handed to the drafter is that of the [SPEC] which follows
        // the accepted path, i.e. the [SPEC] child of its last node (lowest index if several, -1 if none)
        const int win = kMaxNodes - 1 - (s_win & 0xff);
        if (i < n && s_parent[i] == win && s_tok[i] < 0) atomicMin(&s_leaf, i);
        __syncthreads();
        if (i == 0) p.spec_node[b] = s_leaf < kMaxNodes ? s_leaf : -1;
    }
    {
        const int win = kMaxNodes - 1 - (s_win & 0xff);
        const int len = s_win >> 8;
        int32_t* path = p.accept_path + (long long)b * p.path_stride;
        for (int k = len + i; k < p.path_stride; k += blockDim.x) path[k] = -1;     // the padding, all threads
        if (i == 0) {
            p.accept_len[b] = len;
            p.bonus_token[b] = s_am[win];
            int k = len - 1;
            for (int c = win; c >= 0 && k >= 0; c = s_parent[c]) path[k--] = c;
        }
    }
}

// Scan of one (row, vocabulary chunk) item by a single warp: eight 16-byte loads per lane and round.  Per round a
// lane first takes the maximum of its 32 values by a tree of fmaxf (NaN drops out: fmaxf returns the other operand,
// and the final fmaxf with -inf turns an all-NaN round into -inf), and only if that beats its best so far - which
// becomes rare quickly - looks for the first value that attains it.  Strict '>' and first-match keep the lowest
// index among equal values, because a lane's indices grow along its walk; the maximum over (value, ~index) keys
// then does not depend on how the chunk's elements are dealt out to lanes.
// kPipelined: the next round's loads are issued before this round is reduced (twice the registers); the attention
// kernel's guest warps, which run on 72 registers, use the plain form.
template <bool kPipelined>
__device__ __forceinline__ void argmax_scan_chunk_warp(const AcceptParams& p, const int row, const int chunk) {
    const int lane = threadIdx.x & 31;
    const long long V = p.vocab;
    const long long c0 = (long long)chunk * kArgmaxChunk;
    const long long c1 = c0 + kArgmaxChunk < V ? c0 + kArgmaxChunk : V;
    const float* base = p.logits + row * V;
    // [c0, a0) scalar head up to 16-byte alignment, [a0, a1) float4 body, [a1, c1) scalar tail
    const uintptr_t addr = reinterpret_cast<uintptr_t>(base + c0);
    long long a0 = c0 + (long long)(((16 - (addr & 15)) & 15) >> 2);
    if (a0 > c1) a0 = c1;
    const long long a1 = a0 + ((c1 - a0) & ~3ll);

    float bv = -INFINITY;
    uint32_t bi = 0xffffffffu;   // "no candidate yet"
    const float4* body = reinterpret_cast<const float4*>(base + a0);
    const int nvec = (int)((a1 - a0) >> 2);
    const uint64_t policy = l2_evict_first_policy();     // the logits are read once
    const float4 none = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    auto load_round = [&](int v0, float4 (&x)[8]) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {            // eight independent 16-byte loads per lane in flight
            const int v = v0 + j * 32 + lane;
            x[j] = v < nvec ? ld_stream_f4(body + v, policy) : none;
        }
    };
    auto reduce_round = [&](int v0, const float4 (&x)[8]) {
        float m[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) m[j] = fmaxf(fmaxf(x[j].x, x[j].y), fmaxf(x[j].z, x[j].w));
        const float mx = fmaxf(fmaxf(fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3])), fmaxf(fmaxf(m[4], m[5]), fmaxf(m[6], m[7]))), -INFINITY);
        if (v0 + lane < nvec && (bi == 0xffffffffu || mx > bv)) {
            // a new best (or the first candidate): the first of this round's values that attains it; slots past
            // the end hold -inf, which only an all -inf round matches, and then the round's first slot wins
            bv = mx;
#pragma unroll
            for (int j = 7; j >= 0; --j) {
                const uint32_t i0 = (uint32_t)(a0 + 4ll * (v0 + j * 32 + lane));
                if (fmaxf(x[j].w, -INFINITY) == mx) bi = i0 + 3;
                if (fmaxf(x[j].z, -INFINITY) == mx) bi = i0 + 2;
                if (fmaxf(x[j].y, -INFINITY) == mx) bi = i0 + 1;
                if (fmaxf(x[j].x, -INFINITY) == mx) bi = i0;
            }
        }
    };
    if (kPipelined) {
        float4 xa[8], xb[8];
        if (nvec > 0) load_round(0, xa);
        for (int v0 = 0; v0 < nvec; v0 += 2 * 32 * 8) {
            if (v0 + 32 * 8 < nvec) load_round(v0 + 32 * 8, xb);
            reduce_round(v0, xa);
            if (v0 + 2 * 32 * 8 < nvec) load_round(v0 + 2 * 32 * 8, xa);
            if (v0 + 32 * 8 < nvec) reduce_round(v0 + 32 * 8, xb);
        }
    } else {
        for (int v0 = 0; v0 < nvec; v0 += 32 * 8) {
            float4 x[8];
            load_round(v0, x);
            reduce_round(v0, x);
        }
    }
    unsigned long long key = bi != 0xffffffffu ? argmax_key(bv, bi) : 0ull;
    if (lane < 8) {              // ragged ends: at most 3 + 3 elements per chunk
        const long long j = lane < 4 ? c0 + lane : a1 + (lane - 4);
        const long long lim = lane < 4 ? a0 : c1;
        if (j < lim) {
            const unsigned long long k2 = argmax_key(base[j], (uint32_t)j);
            key = k2 > key ? k2 : key;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
        key = other > key ? other : key;
    }
    if (lane == 0) p.part_keys[(long long)row * p.chunks + chunk] = key;
}

// Persistent scan: the grid's warps take the (row, vocabulary chunk) items in turn (consecutive warps read
// consecutive chunks), each with eight 16-byte loads per lane in flight, so that a warp streams without the
// per-item cost of a CTA's launch, barriers and fences.  After storing an item's key, the warp counts it for
// the row's sequence; the warp that counts a sequence's last item notes the sequence, and when the CTA has run
// out of items it walks the trees of the sequences it noted.  (A CTA can note at most as many as it scanned items.)
constexpr int kArgmaxWarps = kArgmaxThreads / 32;
constexpr int kArgmaxCtasPerSm = 2;     // what fits at the kernel's register count
constexpr int kArgmaxNoteMax = 64;
constexpr int kArgmaxOffsMax = 1024;            // sequences whose packed offsets a CTA keeps in shared memory

__global__ void __launch_bounds__(kArgmaxThreads) argmax_partial_kernel(const AcceptParams p) {
    // may be launched as a programmatic dependent of the kernel before it in the stream: nothing is read
    // before that kernel has completed (a no-op in an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may queue up; it waits likewise
    __shared__ int s_note[kArgmaxNoteMax];
    __shared__ int s_notes;
    // packed offsets of up to kArgmaxOffsMax sequences: every item looks its sequence up by binary search, and from
    // global memory that is log2(B) dependent round trips per item with the warp's loads drained
    __shared__ int s_offs[kArgmaxOffsMax + 1];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool offs_staged = p.node_offsets && p.batch <= kArgmaxOffsMax;
    if (offs_staged)
        for (int b = threadIdx.x; b <= p.batch; b += kArgmaxThreads) s_offs[b] = p.node_offsets[b];
    if (threadIdx.x == 0) s_notes = 0;
    if (blockIdx.x == 0) {
        // Once per call: clear every counter of the idle set (the next call counts there, whatever its batch), and
        // check that the packed offsets describe this call's rows: start at 0, end at total_nodes, 1..max_nodes
        // nodes per sequence.  With inconsistent offsets a row would count for the wrong sequence and a walk could
        // run on keys not yet stored; the status word says so (that call's outputs are then meaningless).
        unsigned int* idle = p.seq_counter + (size_t)((p.epoch + 1u) & 1u) * p.counter_stride;
        for (int b = threadIdx.x; b < p.counter_stride; b += kArgmaxThreads) idle[b] = 0u;
        if (p.node_offsets) {
            bool bad = false;
            for (int b = threadIdx.x; b < p.batch; b += kArgmaxThreads) {
                const int lo = p.node_offsets[b], n = p.node_offsets[b + 1] - lo;
                bad = bad || n < 1 || n > p.max_nodes || (b == 0 && lo != 0) || (b == p.batch - 1 && lo + n != p.total_nodes);
            }
            if (bad) report(p.status, kErrBadTree);
        }
    }
    __syncthreads();
    const long long items = (long long)p.total_nodes * p.chunks;
    const long long stride = (long long)gridDim.x * kArgmaxWarps;
    for (long long it = (long long)blockIdx.x * kArgmaxWarps + warp; it < items; it += stride) {
        const int row = (int)(it / p.chunks), chunk = (int)(it - (long long)row * p.chunks);
        argmax_scan_chunk_warp<true>(p, row, chunk);
        if (lane == 0) {
            // which sequence owns this row, and is this the last of its chunk keys?
            int b, n_b;
            if (p.node_offsets) {
                const int* offs = offs_staged ? s_offs : p.node_offsets;
                int lo = 0, hi = p.batch;   // largest b with node_offsets[b] <= row
                while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (offs[mid] <= row) lo = mid; else hi = mid; }
                b = lo;
                n_b = offs[b + 1] - offs[b];
            } else {
                b = row / p.nodes_uniform;
                n_b = p.nodes_uniform;
            }
            __threadfence();
            // two sets of counters: this call counts in set (epoch & 1); the other one is cleared as a whole (above)
            // for the next call, so a counter left dirty by malformed input is gone two calls later at the latest and
            // is never counted in
            unsigned int* ctr = p.seq_counter + (size_t)(p.epoch & 1u) * p.counter_stride + b;
            const unsigned int want = atomicAdd(ctr, 1u) + 1u;
            if ((long long)want == (long long)p.chunks * n_b) {
                *ctr = 0u;                                   // a completed counter is left clean as well
                const int slot = atomicAdd(&s_notes, 1);
                if (slot < kArgmaxNoteMax) s_note[slot] = b;
                else report(p.status, kErrBadTree);          // only inconsistent offsets can complete that many here
            }
        }
    }
    __threadfence();
    __syncthreads();
    const int notes = min(s_notes, kArgmaxNoteMax);
    for (int k = 0; k < notes; ++k) {
        accept_walk_seq(p, s_note[k]);
        __syncthreads();
    }
}

// Grid of the scan for `items` (row, chunk) items on a device with `sms` multiprocessors: as many warps as give
// every warp the same number of items (4096 items on 2368 resident warps would leave a quarter of the warps idle
// during the second half of the kernel; 2048 warps with two items each do not).
__host__ inline unsigned argmax_grid(long long items, int sms) {
    const long long max_warps = (long long)sms * kArgmaxCtasPerSm * kArgmaxWarps;
    const long long rounds = (items + max_warps - 1) / max_warps;
    const long long warps = rounds > 0 ? (items + rounds - 1) / rounds : 1;
    const long long ctas = (warps + kArgmaxWarps - 1) / kArgmaxWarps;
    return (unsigned)(ctas < 1 ? 1 : ctas);
}

}  // namespace owl
