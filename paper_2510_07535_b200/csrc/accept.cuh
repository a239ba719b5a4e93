// Greedy tree acceptance: row arg-max over the vocabulary, then the acceptance walk.
//
// Kernel 1 scans fp32 logits with 16-byte loads.  Every (value, index) candidate is folded into
// one 64-bit key, high word = the float mapped to an unsigned integer that sorts like the float
// (NaN mapped to -inf, -0 to +0), low word = ~index, so that an unsigned max picks the larger
// value and, among equal values, the lower index.  Per-thread, warp (shuffle) and block maxima
// give one key per (row, vocabulary chunk), stored to part_keys[row][chunk] (no atomics, nothing
// to initialise).
//
// The CTA that stores the last chunk key of a sequence (a per-sequence counter, bumped after a
// __threadfence; nobody waits for anybody) then does that sequence's walk in the same launch: it reduces
// the chunk keys to arg-max tokens, evaluates for every node whether all edges on its root path match
// (draft token == parent's arg-max), picks the deepest matching node (lowest index among equals) and
// writes accept_len / accept_path / bonus_token.  Calls alternate between two sets of counters and clear the
// idle one as a whole, so no separate clearing pass is needed.
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
static_assert(kArgmaxChunk == 8 * 4 * kArgmaxThreads, "argmax_partial_kernel reads its chunk in one round of 8 loads");

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
    if (i == 0) {
        const int win = kMaxNodes - 1 - (s_win & 0xff);
        const int len = s_win >> 8;
        p.accept_len[b] = len;
        p.bonus_token[b] = s_am[win];
        int32_t* path = p.accept_path + (long long)b * p.path_stride;
        for (int k = len; k < p.path_stride; ++k) path[k] = -1;
        int k = len - 1;
        for (int c = win; c >= 0 && k >= 0; c = s_parent[c]) path[k--] = c;
    }
}

// The same scan of one (row, vocabulary chunk) by a single warp, for callers that have warps to spare inside
// another kernel (the verify step's attention pass scans the logits with its two idle warps while it streams K/V).
// Stores the same key argmax_partial_kernel would: the maximum over (value, ~index) does not depend on how the
// chunk's elements are dealt out to threads.
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
    for (int v0 = 0; v0 < nvec; v0 += 32 * 8) {
        float4 x[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {            // eight independent 16-byte loads per lane in flight
            const int v = v0 + j * 32 + lane;
            x[j] = v < nvec ? __ldg(body + v) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int v = v0 + j * 32 + lane;
            if (v < nvec) {
                const uint32_t i0 = (uint32_t)(a0 + 4ll * v);
                // NaN reads as -inf; strict '>' keeps the first maximum (indices grow along this lane's walk)
                const float e0 = x[j].x != x[j].x ? -INFINITY : x[j].x, e1 = x[j].y != x[j].y ? -INFINITY : x[j].y;
                const float e2 = x[j].z != x[j].z ? -INFINITY : x[j].z, e3 = x[j].w != x[j].w ? -INFINITY : x[j].w;
                if (bi == 0xffffffffu || e0 > bv) { bv = e0; bi = i0; }
                if (e1 > bv) { bv = e1; bi = i0 + 1; }
                if (e2 > bv) { bv = e2; bi = i0 + 2; }
                if (e3 > bv) { bv = e3; bi = i0 + 3; }
            }
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

__global__ void __launch_bounds__(kArgmaxThreads) argmax_partial_kernel(const AcceptParams p) {
    // may be launched as a programmatic dependent of the kernel before it in the stream: nothing is read
    // before that kernel has completed (a no-op in an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may queue up; it waits likewise
    const int row = blockIdx.y;
    if (blockIdx.x == 0 && blockIdx.y == 0) {
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
    const long long V = p.vocab;
    const long long c0 = (long long)blockIdx.x * kArgmaxChunk;
    const long long c1 = c0 + kArgmaxChunk < V ? c0 + kArgmaxChunk : V;
    const float* base = p.logits + row * V;

    // [c0, a0) scalar head up to 16-byte alignment, [a0, a1) float4 body, [a1, c1) scalar tail
    const uintptr_t addr = reinterpret_cast<uintptr_t>(base + c0);
    long long a0 = c0 + (long long)(((16 - (addr & 15)) & 15) >> 2);
    if (a0 > c1) a0 = c1;
    const long long a1 = a0 + ((c1 - a0) & ~3ll);

    float bv = -INFINITY;
    uint32_t bi = 0xffffffffu;   // "no candidate yet"
    unsigned long long key = 0;
    const float4* body = reinterpret_cast<const float4*>(base + a0);
    const int nvec = (int)((a1 - a0) >> 2);
    // A chunk is 8 x 16 bytes per thread: all eight loads are issued before the first compare, so that a CTA has its
    // whole 32 KB in flight at once (one load per iteration left the scan at about half of the memory bandwidth).
    // The logits are read once: they bypass L1 and are the first to leave L2.
    {
        const uint64_t policy = l2_evict_first_policy();
        float4 x[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int v = j * kArgmaxThreads + (int)threadIdx.x;
            x[j] = v < nvec ? ld_stream_f4(body + v, policy) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int v = j * kArgmaxThreads + (int)threadIdx.x;
            if (v < nvec) {
                const uint32_t i0 = (uint32_t)(a0 + 4ll * v);
                // NaN reads as -inf; strict '>' keeps the first maximum (indices grow along this thread's walk)
                const float e0 = x[j].x != x[j].x ? -INFINITY : x[j].x, e1 = x[j].y != x[j].y ? -INFINITY : x[j].y;
                const float e2 = x[j].z != x[j].z ? -INFINITY : x[j].z, e3 = x[j].w != x[j].w ? -INFINITY : x[j].w;
                if (bi == 0xffffffffu || e0 > bv) { bv = e0; bi = i0; }
                if (e1 > bv) { bv = e1; bi = i0 + 1; }
                if (e2 > bv) { bv = e2; bi = i0 + 2; }
                if (e3 > bv) { bv = e3; bi = i0 + 3; }
            }
        }
    }
    if (bi != 0xffffffffu) key = argmax_key(bv, bi);
    // ragged ends: at most 3 + 3 elements per chunk
    if (threadIdx.x < 8) {
        long long j = threadIdx.x < 4 ? c0 + threadIdx.x : a1 + (threadIdx.x - 4);
        const long long lim = threadIdx.x < 4 ? a0 : c1;
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
    __shared__ unsigned long long s_key[kArgmaxThreads / 32];
    if ((threadIdx.x & 31) == 0) s_key[threadIdx.x >> 5] = key;
    __syncthreads();
    __shared__ int s_walk_b;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 1; w < kArgmaxThreads / 32; ++w) key = s_key[w] > key ? s_key[w] : key;
        p.part_keys[(long long)row * p.chunks + blockIdx.x] = key;
        // which sequence owns this row, and is this the last of its chunk keys?
        int b, n_b;
        if (p.node_offsets) {
            int lo = 0, hi = p.batch;   // largest b with node_offsets[b] <= row
            while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (p.node_offsets[mid] <= row) lo = mid; else hi = mid; }
            b = lo;
            n_b = p.node_offsets[b + 1] - p.node_offsets[b];
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
        if ((long long)want == (long long)p.chunks * n_b) *ctr = 0u;   // a completed counter is left clean as well
        s_walk_b = ((long long)want == (long long)p.chunks * n_b) ? b : -1;
        __threadfence();
    }
    __syncthreads();
    if (s_walk_b >= 0) accept_walk_seq(p, s_walk_b);
}

}  // namespace owl
