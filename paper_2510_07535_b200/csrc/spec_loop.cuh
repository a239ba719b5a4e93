// The steps of the decoding loop on either side of the verify pass (Algorithm 1):
//   prepare_spec_kernel   Prepare(d): one [SPEC] leaf after every tree path, parents (= attention mask),
//                         depth-based position ids (Section 3.2.2 "Decode Stage")
//   kv_commit_*_kernel    "l <- l; d", "N <- N + |d|": the accepted nodes' K/V move from logical position
//                         L + path[k] to L + k in the paged cache, the committed length grows by accept_len
// Both are tiny and latency-bound: one CTA per sequence (and per KV head and cache for the move).
#pragma once

#include "owl_common.cuh"

namespace owl {

struct PrepareParams {
    const int32_t* node_offsets;   // may be null: nodes_uniform drafted nodes per sequence
    const int32_t* tree_parent;
    const int32_t* draft_tokens;
    const int32_t* ctx_lens;
    const int32_t* route;          // may be null (every sequence gets [SPEC] leaves); route[b] == 0: chain kept as drafted
    int32_t* out_offsets;          // [B + 1]: running sum of the output node counts (n or 2 n per sequence)
    int32_t* out_parent;           // [2 N]
    int32_t* out_draft;            // [2 N], -1 for a [SPEC] leaf
    int32_t* out_input_ids;        // [2 N], spec_token for a [SPEC] leaf
    int32_t* out_position;         // [2 N], ctx_len + depth
    int32_t* status;
    int32_t batch, total_nodes, nodes_uniform, max_nodes, spec_token;
};

constexpr int kPrepareThreads = 64;
static_assert(kPrepareThreads >= kMaxNodes, "one thread per drafted node");

// One CTA per sequence, one thread per drafted node j: node j keeps its place, its [SPEC] leaf is node n + j.
// With a route array, a sequence routed to non-tree verification (route 0) keeps its chain without any [SPEC]
// (Section 3.2.3); the sequences' outputs are packed one after the other, so every CTA first sums the output
// node counts of the sequences before its own.
__global__ void __launch_bounds__(kPrepareThreads) prepare_spec_kernel(const PrepareParams p) {
    // may be launched as a programmatic dependent: nothing is read before the kernel before it in the stream has
    // completed (a no-op in an ordinary launch); the kernel after this one may queue up and waits likewise
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int b = blockIdx.x, j = threadIdx.x;
    const int base = p.node_offsets ? p.node_offsets[b] : b * p.nodes_uniform;
    const int n = p.node_offsets ? p.node_offsets[b + 1] - base : p.nodes_uniform;
    const bool with_spec = !p.route || p.route[b] != 0;
    __shared__ int s_parent[kMaxNodes];
    __shared__ int s_bad, s_before;
    if (j == 0) { s_bad = 0; s_before = 0; }
    __syncthreads();
    long long before = 0;            // output nodes of sequences 0 .. b-1
    if (p.route) {
        for (int c = j; c < b; c += kPrepareThreads) {
            const int nc = p.node_offsets ? p.node_offsets[c + 1] - p.node_offsets[c] : p.nodes_uniform;
            before += p.route[c] != 0 ? 2 * nc : nc;
        }
        atomicAdd(&s_before, (int)before);
    } else if (j == 0) {
        s_before = 2 * base;
    }
    __syncthreads();
    const int ob = s_before, count = with_spec ? 2 * n : n;
    if (j == 0) {
        // the outputs hold 2 * total_nodes entries: whatever the offsets say, nothing is written outside them
        s_bad = (n < 1 || n > p.max_nodes || count > kMaxNodes || base < 0 || base + n > p.total_nodes || ob < 0 ||
                 (long long)ob + count > 2ll * p.total_nodes) ? 1 : 0;
        if (b == 0) p.out_offsets[0] = 0;
        p.out_offsets[b + 1] = ob + count;
    }
    __syncthreads();
    if (s_bad) { if (j == 0) report(p.status, kErrBadTree); return; }
    int parent = -1;
    if (j < n) {
        parent = p.tree_parent[base + j];
        s_parent[j] = parent;
        if ((j == 0 && parent != -1) || (j > 0 && (parent < 0 || parent >= j))) atomicExch(&s_bad, 1);
    }
    __syncthreads();
    if (s_bad) { if (j == 0) report(p.status, kErrBadTree); return; }   // nothing of this sequence is written
    if (j < n) {
        int depth = 0;
        for (int c = j; s_parent[c] >= 0 && depth < kMaxNodes; c = s_parent[c]) ++depth;
        const int L = p.ctx_lens[b], tok = p.draft_tokens[base + j];
        const int o = ob + j;
        p.out_parent[o] = parent;
        p.out_draft[o] = tok;
        p.out_input_ids[o] = tok;
        p.out_position[o] = L + depth;
        if (with_spec) {
            p.out_parent[o + n] = j;
            p.out_draft[o + n] = -1;
            p.out_input_ids[o + n] = p.spec_token;
            p.out_position[o + n] = L + depth + 1;
        }
    }
}

struct CommitParams {
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
    const int32_t* block_table;
    int32_t* ctx_lens;             // in / out
    const int32_t* node_offsets;   // may be null
    const int32_t* accept_len;
    const int32_t* accept_path;
    int32_t* status;
    int32_t batch, total_nodes, nodes_uniform, max_nodes, num_kv_heads;
    int32_t page_size, page_shift, max_pages_per_seq, num_pages, path_stride;
};

constexpr int kCommitThreads = 256;

// What both commit kernels decide alike for sequence b, from the inputs alone: 0 = commit, else the error code.
// The accepted path must be a root path in node order (path[0] = 0, strictly increasing, below n) and every page
// the drafted positions L .. L + n - 1 touch must exist.  Called by all threads of a CTA (uses two barriers).
__device__ __forceinline__ int commit_verdict(const CommitParams& p, int b, int& L, int& n, int& a, int* s_path /*[kMaxNodes]*/,
                                              int* s_flag) {
    const int base = p.node_offsets ? p.node_offsets[b] : b * p.nodes_uniform;
    n = p.node_offsets ? p.node_offsets[b + 1] - base : p.nodes_uniform;
    L = p.ctx_lens[b];
    a = p.accept_len[b];
    if (threadIdx.x == 0) *s_flag = 0;
    __syncthreads();
    const bool shape_ok = n >= 1 && n <= p.max_nodes && n <= kMaxNodes && a >= 1 && a <= n && a <= p.path_stride && L >= 0 &&
                          (long long)L + n <= (long long)p.max_pages_per_seq * p.page_size;
    if (!shape_ok) return kErrBadTree;
    const int t = threadIdx.x;
    if (t < a) {
        const int v = p.accept_path[(long long)b * p.path_stride + t];
        s_path[t] = v;
        const int prev = t > 0 ? p.accept_path[(long long)b * p.path_stride + t - 1] : -1;
        if ((t == 0 && v != 0) || v <= prev || v >= n) atomicExch(s_flag, kErrBadTree);
    }
    const int first_page = L >> p.page_shift, last_page = (L + n - 1) >> p.page_shift;
    if (t <= last_page - first_page) {
        const int pg = p.block_table[(long long)b * p.max_pages_per_seq + first_page + t];
        if ((unsigned)pg >= (unsigned)p.num_pages) atomicCAS(s_flag, 0, kErrBadPage);
    }
    __syncthreads();
    return *s_flag;
}

// grid (2 * Hkv, B): blockIdx.x = 2 * head + (0: K, 1: V).  Every source row is read into shared memory before any
// destination is written, because a position can be the source of one move and the destination of a later one.
__global__ void __launch_bounds__(kCommitThreads) kv_commit_move_kernel(const CommitParams p) {
    // may be launched as a programmatic dependent: nothing is read before the kernel before it in the stream has
    // completed (a no-op in an ordinary launch); the kernel after this one may queue up and waits likewise
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ uint4 s_rows[kMaxNodes * 16];       // up to 64 rows of 128 bf16
    __shared__ int s_path[kMaxNodes];
    __shared__ int s_flag;
    const int b = blockIdx.y, h = blockIdx.x >> 1;
    int L, n, a;
    const int verdict = commit_verdict(p, b, L, n, a, s_path, &s_flag);
    if (verdict != 0) {
        if (threadIdx.x == 0 && blockIdx.x == 0) report(p.status, verdict);
        return;
    }
    __nv_bfloat16* cache = (blockIdx.x & 1) ? p.v_cache : p.k_cache;
    const int32_t* table = p.block_table + (long long)b * p.max_pages_per_seq;
    auto row_ptr = [&](int pos) {
        const long long page = table[pos >> p.page_shift];
        return reinterpret_cast<uint4*>(cache + ((page * p.num_kv_heads + h) * p.page_size + (pos & (p.page_size - 1))) * kHeadDim);
    };
    const int piece = threadIdx.x & 15;
    for (int k = threadIdx.x >> 4; k < a; k += kCommitThreads / 16)
        if (s_path[k] != k) s_rows[k * 16 + piece] = row_ptr(L + s_path[k])[piece];
    __syncthreads();
    for (int k = threadIdx.x >> 4; k < a; k += kCommitThreads / 16)
        if (s_path[k] != k) row_ptr(L + k)[piece] = s_rows[k * 16 + piece];
}

// One CTA per sequence, after the move kernel in stream order: the committed length grows by accept_len.
__global__ void __launch_bounds__(kCommitThreads) kv_commit_lens_kernel(const CommitParams p) {
    // may be launched as a programmatic dependent: nothing is read before the kernel before it in the stream has
    // completed (a no-op in an ordinary launch); the kernel after this one may queue up and waits likewise
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ int s_path[kMaxNodes];
    __shared__ int s_flag;
    int L, n, a;
    const int verdict = commit_verdict(p, blockIdx.x, L, n, a, s_path, &s_flag);
    if (verdict == 0 && threadIdx.x == 0) p.ctx_lens[blockIdx.x] = L + a;
}

}  // namespace owl
