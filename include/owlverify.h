/*
 * libowlverify - the target model's verification step of long-context speculative
 * decoding (OWL / HOWL), for one NVIDIA B200 (sm_100a).
 *
 * Two operations, as the paper states the problem:
 *   owl_verify_attn  - every drafted token (a chain, or a token tree with [SPEC]
 *                      leaves) attends to the whole cached context plus the nodes on
 *                      its own root path, all nodes in one pass (Introduction;
 *                      Section 3.2.2 "Decode Stage": attention mask manipulated so that
 *                      each appended token follows exactly one tree path; Section 3.2.3 /
 *                      Algorithm 1: NonTreeVerify is the same pass on a chain).
 *   owl_tree_accept  - the decoding algorithm then accepts the drafted tokens that keep
 *                      the target's output distribution (Introduction); under greedy
 *                      decoding: per-node arg-max over the vocabulary, the longest root
 *                      path whose drafted tokens equal their parent's arg-max, and the
 *                      arg-max of the last accepted node as the next token.  The number
 *                      of tokens accepted per step is the paper's "acceptance length"
 *                      (Figure 1 caption), at least 1 and at most tree depth + 1
 *                      (Appendix "Inference Details": depth 8, maximum 9).
 *
 * General rules of this interface
 *  - Plain C ABI.  Unless an argument says "host", every tensor pointer is a DEVICE
 *    pointer on the context's device, owned by the caller; the library reads inputs,
 *    writes outputs, and neither frees nor keeps any of them after the call's work
 *    has run on the stream.
 *  - Calls enqueue work on the caller's stream (a cudaStream_t passed as void*;
 *    NULL = the default stream) and return without synchronising the host, except
 *    owl_get_status and the *_host convenience call, which synchronise that stream.
 *  - Return value: OWL_OK or a negative owl_status.  Errors that can be seen from the
 *    arguments alone are returned immediately and launch nothing.  Errors that need
 *    device data (a malformed tree, a page id out of range) are recorded in a device
 *    status word read by owl_get_status; the kernels then leave the outputs of the
 *    offending sequence unwritten and finish normally.
 *  - One owl_ctx serves one stream at a time (its workspace is reused by every call).
 *
 * Layouts (B sequences, N = total drafted nodes packed sequence after sequence,
 * Hq query heads, Hkv key/value heads, G = Hq/Hkv, D = head_dim = 128):
 *  - q, out       bf16 [N, Hq, D]
 *  - lse          fp32 [N, Hq]   natural log of sum_k exp(sm_scale * q.k) over visible keys
 *  - k_cache/v_cache  bf16 [num_pages, Hkv, page_size, D]; one (page, head) block is
 *                 page_size*D contiguous elements.  A contiguous cache is the same
 *                 layout with an identity block_table.
 *  - block_table  int32 [B, max_pages_per_seq]: physical page of each logical page
 *  - ctx_lens     int32 [B]: committed context length L_b.  The K/V of drafted node i
 *                 of sequence b are already stored at logical position L_b + i, so the
 *                 cache holds L_b + n_b valid positions.  Q and K arrive with their
 *                 rotary position (the paper's position-id manipulation) applied.
 *                 Cache slots of a sequence's last page beyond L_b + n_b are never
 *                 visible and may hold anything (uninitialised memory, NaN, Inf).
 *  - node_offsets int32 [B+1], packed offsets of each sequence's nodes; NULL means
 *                 every sequence has N/B nodes.
 *  - tree_parent  int32 [N]: parent of each node as an index local to its sequence,
 *                 -1 for the root.  Node 0 of a sequence is its only root and
 *                 parent[i] < i (topological / BFS order).  The root is the target's own
 *                 already chosen token t_{N+1}.
 */
#ifndef OWLVERIFY_H_
#define OWLVERIFY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum owl_status {
    OWL_OK = 0,
    OWL_ERR_INVALID_ARG = -1, /* null pointer, batch < 1, total_nodes < 1, Hq % Hkv != 0, ...       */
    OWL_ERR_UNSUPPORTED = -2, /* head_dim != 128, max_nodes > 64, G*max_nodes > 256, page size, ... */
    OWL_ERR_CUDA = -3,        /* a CUDA call failed; see owl_last_error                             */
    OWL_ERR_BAD_TREE = -4,    /* device-detected: parent[i] >= i, parent < -1, node 0 not the root,
                                 a sequence with no or too many nodes, inconsistent node_offsets    */
    OWL_ERR_BAD_PAGE = -5,    /* device-detected: block_table entry outside [0, num_pages)          */
    OWL_ERR_TIMEOUT = -6,     /* device-detected: a bounded wait inside a kernel expired            */
    OWL_ERR_TOO_LARGE = -7    /* dims exceed what the context was created for                       */
} owl_status;

typedef struct owl_ctx owl_ctx; /* opaque: device workspace (split partials, status word) */

typedef struct owl_dims {
    int32_t batch;             /* B >= 1                                                        */
    int32_t total_nodes;       /* N = sum of n_b >= B                                           */
    int32_t max_nodes;         /* T = max n_b, 1..64 (the paper's trees have 60 nodes)          */
    int32_t num_q_heads;       /* Hq                                                            */
    int32_t num_kv_heads;      /* Hkv <= 128, divides Hq; G*T <= 256                            */
    int32_t head_dim;          /* must be 128                                                   */
    int32_t page_size;         /* tokens per page: 16 (also 32, 64, 128)                        */
    int32_t max_pages_per_seq; /* row stride of block_table                                     */
    int32_t num_pages;         /* pages in k_cache / v_cache; block_table entries are checked   */
    int32_t vocab;             /* V (owl_tree_accept only; may be 0 for attention-only use)     */
    int32_t path_stride;       /* row stride of accept_path, >= max_nodes (64 always is)        */
    float sm_scale;            /* multiplies q.k before the softmax; explicit, finite, > 0      */
} owl_dims;

/* Create a context on `device` with workspace for any call whose dims do not exceed
 * `max_dims` (batch, total_nodes, max_nodes, heads).  Allocates device memory once;
 * later calls allocate nothing.  Host-synchronous. */
int owl_create(owl_ctx** ctx, int device, const owl_dims* max_dims);

/* Free the context's device memory.  The caller must have synchronised every stream
 * that used it. */
int owl_destroy(owl_ctx* ctx);

/*
 * Tree-masked attention of the drafted nodes against the paged KV cache
 * (Section 3.2.2 "Decode Stage"; Algorithm 1, NonTreeVerify / OurTreeVerify).
 *
 * For packed node n = node_offsets[b] + i and query head hq (KV head hq / G):
 *   visible keys = {0 .. L_b-1}  union  {L_b + j : j on the root path of i, i included}
 *   out[n,hq,:]  = sum_k softmax_k(sm_scale * q[n,hq].K_k) * V_k   (rounded to bf16)
 *   lse[n,hq]    = ln sum_k exp(sm_scale * q[n,hq].K_k)
 * Computed by split-KV kernels: per KV chunk an online-softmax pass on the tensor
 * cores producing fp32 partials in the context's workspace, then an LSE merge.
 * Asynchronous on `stream`.  `lse` may be NULL.
 */
int owl_verify_attn(owl_ctx* ctx, const owl_dims* dims, const void* q, const void* k_cache,
                    const void* v_cache, const int32_t* block_table, const int32_t* ctx_lens,
                    const int32_t* node_offsets, const int32_t* tree_parent, void* out, float* lse,
                    void* stream);

/*
 * owl_verify_attn with q, k_cache, v_cache and out in fp16 (IEEE binary16) instead of bf16: the data type the
 * paper ran in (Appendix "Inference Details": "use fp16 data type").  Same layouts, same semantics, same
 * tolerances; the softmax weights are rounded to fp16 before the second product, lse stays fp32.
 */
int owl_verify_attn_f16(owl_ctx* ctx, const owl_dims* dims, const void* q, const void* k_cache,
                        const void* v_cache, const int32_t* block_table, const int32_t* ctx_lens,
                        const int32_t* node_offsets, const int32_t* tree_parent, void* out, float* lse,
                        void* stream);

/*
 * Greedy tree acceptance (Introduction: accepted tokens keep the target's output
 * distribution; Figure 1 caption: acceptance length; Section 3.2.2: paths start at the
 * root t_{N+1}, [SPEC] leaves are never candidate tokens).
 *
 *   am[n]      = lowest index attaining the maximum of logits[n, :] (NaN reads as -inf)
 *   ok(root)   = true;  ok(i) = ok(parent(i)) and draft_tokens[i] >= 0
 *                              and draft_tokens[i] == am[parent(i)]
 *   winner     = ok node of greatest depth, lowest index among equals
 *   accept_len[b]    = depth(winner) + 1            (nodes on the path, root included)
 *   accept_path[b,:] = local node indices root..winner, then -1 up to path_stride
 *   bonus_token[b]   = am[winner]                   (the target's next token)
 *
 * logits fp32 [N, V] row-major (row n = packed node n); draft_tokens int32 [N]
 * (the root's entry is ignored; a negative entry, e.g. a [SPEC] leaf, never matches);
 * node_argmax optional int32 [N] (NULL to skip) receives am.  Asynchronous on `stream`.
 */
int owl_tree_accept(owl_ctx* ctx, const owl_dims* dims, const float* logits,
                    const int32_t* draft_tokens, const int32_t* node_offsets,
                    const int32_t* tree_parent, int32_t* accept_len, int32_t* accept_path,
                    int32_t* bonus_token, int32_t* node_argmax, void* stream);

/*
 * owl_tree_accept with one more output for trees that carry [SPEC] leaves (Section 3.2.2 "Decode Stage":
 * "when a path is accepted, we take the hidden state of the corresponding [SPEC]"; Algorithm 1, h_S returned
 * by OurTreeVerify): spec_node[b] (device int32 [B], required) = local index of the [SPEC] leaf - a child with
 * a negative draft token - of the last node of the accepted path, the lowest index if there are several, -1 if
 * that node has none (a chain verified without [SPEC]).  Everything else as owl_tree_accept.
 */
int owl_tree_accept_spec(owl_ctx* ctx, const owl_dims* dims, const float* logits,
                         const int32_t* draft_tokens, const int32_t* node_offsets,
                         const int32_t* tree_parent, int32_t* accept_len, int32_t* accept_path,
                         int32_t* bonus_token, int32_t* spec_node, int32_t* node_argmax, void* stream);

/*
 * Prepare(d) of Algorithm 1 (Section 3.2.2 "Decode Stage"): appends one [SPEC] token after every tree path - as
 * many [SPEC] as the drafted tree has nodes - and derives what the verifier needs: the parents (from which
 * owl_verify_attn builds the attention mask) and the manipulated position ids.
 *
 * In (device): the drafted trees as for owl_verify_attn (dims->batch, dims->total_nodes, dims->max_nodes <= 32;
 * node_offsets [B+1] or NULL for uniform; tree_parent [N]; draft_tokens [N], the root's entry being the target's
 * own token t_{N+1}); ctx_lens [B]; spec_token = token id of [SPEC].
 * Out (device, caller-owned), sequence b with n nodes occupying [2*node_offsets[b], 2*node_offsets[b] + 2n):
 *   out_node_offsets [B+1]  = 2 * node_offsets
 *   out_tree_parent  [2N]   nodes 0..n-1 as drafted; node n + j is the [SPEC] after the path ending in node j
 *   out_draft_tokens [2N]   drafted token; -1 for a [SPEC] leaf (never a candidate of the acceptance)
 *   out_input_ids    [2N]   what the verifier embeds: drafted token; spec_token for a leaf
 *   out_position_ids [2N]   ctx_lens[b] + depth of the node (root: depth 0)
 * The prepared trees (2n <= 64 nodes, parent[i] < i) go to owl_verify_attn / owl_tree_accept_spec with
 * total_nodes = 2N, max_nodes = 2 * dims->max_nodes.  Asynchronous on `stream`.  A malformed tree sets
 * OWL_ERR_BAD_TREE in the status word and leaves that sequence's rows unwritten.
 */
int owl_prepare_spec_tree(owl_ctx* ctx, const owl_dims* dims, const int32_t* node_offsets,
                          const int32_t* tree_parent, const int32_t* draft_tokens, const int32_t* ctx_lens,
                          int32_t spec_token, int32_t* out_node_offsets, int32_t* out_tree_parent,
                          int32_t* out_draft_tokens, int32_t* out_input_ids, int32_t* out_position_ids,
                          void* stream);

/*
 * The routing decision of Algorithm 1 (Section 3.2.3), once per sequence and decoding step.  HOST arrays: the
 * score comes from the non-tree drafter, which runs on the CPU, and the decision steers host control flow
 * (which drafter runs next).  score[b] = that drafter's estimate of its acceptance length; c = the threshold
 * (the paper uses 9, the longest acceptance its depth-8 trees allow, Appendix "Inference Details");
 * lastwaslinear[b] (in/out, 0 before the first step) = whether the sequence's previous step was verified as a
 * chain.  route[b] (out):
 *   OWL_ROUTE_LINEAR       score > c: verify the non-tree drafter's chain as drafted, no [SPEC] appended
 *   OWL_ROUTE_TREE_NOSPEC  score <= c after a linear step: tree from the drafter trained without [SPEC]
 *                          (the linear step produced no [SPEC] hidden state)
 *   OWL_ROUTE_TREE_SPEC    score <= c otherwise: tree from the drafter trained with [SPEC]
 * Both tree routes are verified with [SPEC] leaves (owl_prepare_hybrid).  A NaN score takes a tree route.
 * Returns OWL_ERR_INVALID_ARG for batch < 1, a NULL pointer or a NaN threshold.
 */
#define OWL_ROUTE_LINEAR 0
#define OWL_ROUTE_TREE_NOSPEC 1
#define OWL_ROUTE_TREE_SPEC 2
int owl_howl_route(int32_t batch, const float* score, float c, uint8_t* lastwaslinear, int32_t* route);

/*
 * Prepare(d) on a routed batch (Algorithm 1; Section 3.2.3: on the non-tree route "we do not append any [SPEC]").
 * As owl_prepare_spec_tree, with route (device int32 [B], the values owl_howl_route gives): a sequence with
 * route OWL_ROUTE_LINEAR keeps its n nodes as drafted (position ids ctx_len + depth, input ids = tokens), every
 * other sequence becomes 2n nodes with [SPEC] leaves.  The sequences' outputs are packed one after the other:
 * out_node_offsets [B+1] is the running sum of n or 2n; the other outputs need room for 2 * total_nodes entries.
 * dims->max_nodes bounds the DRAFTED nodes of a sequence: up to 64 on the linear route, up to 32 on a tree route
 * (a longer tree sets OWL_ERR_BAD_TREE on the device and leaves that sequence unwritten).
 */
int owl_prepare_hybrid(owl_ctx* ctx, const owl_dims* dims, const int32_t* node_offsets,
                       const int32_t* tree_parent, const int32_t* draft_tokens, const int32_t* ctx_lens,
                       const int32_t* route, int32_t spec_token, int32_t* out_node_offsets,
                       int32_t* out_tree_parent, int32_t* out_draft_tokens, int32_t* out_input_ids,
                       int32_t* out_position_ids, void* stream);

/*
 * Commit of the accepted tokens to the cache (Algorithm 1: "l <- l; d", "N <- N + |d|").  During verification
 * the K/V of drafted node i of sequence b sit at logical position L_b + i; for the accepted path p_0 = 0 < p_1 <
 * ... < p_{a-1} (accept_path / accept_len as owl_tree_accept wrote them) the rows at L_b + p_k move to L_b + k,
 * for every KV head, in k_cache and v_cache, IN PLACE, and ctx_lens[b] becomes L_b + a.  Whatever else was
 * drafted stays behind as dead slots past the new length.  Uses dims->batch, total_nodes, max_nodes,
 * num_kv_heads, head_dim, page_size, max_pages_per_seq, num_pages, path_stride.  All pointers device; k_cache,
 * v_cache and ctx_lens are read and written.  Asynchronous on `stream` (two small kernels in stream order).  A
 * path that is not a root path in node order sets OWL_ERR_BAD_TREE, a page id out of range OWL_ERR_BAD_PAGE;
 * that sequence is then left untouched, length included.
 */
int owl_kv_commit(owl_ctx* ctx, const owl_dims* dims, void* k_cache, void* v_cache,
                  const int32_t* block_table, int32_t* ctx_lens, const int32_t* node_offsets,
                  const int32_t* accept_len, const int32_t* accept_path, void* stream);

/*
 * Acceptance straight from the verifier's last hidden states (Introduction: the target model's forward over the
 * drafted tokens ends in logits, from which the accepted tokens follow): logits[n, :] = hidden[n, :] . weight^T is
 * computed on the tensor cores (bf16 operands, fp32 accumulation) and reduced to its row arg-max inside the same
 * kernel - the [N, V] logits are never written - then the acceptance walk of owl_tree_accept runs on those arg-max
 * tokens.  hidden bf16 [N, hidden_dim] (row n = packed node n), weight bf16 [V, hidden_dim] (the LM head,
 * output-major); hidden_dim a multiple of 64; N = dims->total_nodes <= 384; V = dims->vocab.  The other arguments
 * and all outputs as owl_tree_accept.  Two logits of a row that differ by less than what fp32 accumulation order
 * can move them (about 1e-5 for unit-scale operands) may be ranked either way; exact ties go to the lower index.
 * Asynchronous on `stream`; device pointers, caller-owned.
 */
int owl_lm_head_accept(owl_ctx* ctx, const owl_dims* dims, int32_t hidden_dim, const void* hidden,
                       const void* weight, const int32_t* draft_tokens, const int32_t* node_offsets,
                       const int32_t* tree_parent, int32_t* accept_len, int32_t* accept_path,
                       int32_t* bonus_token, int32_t* node_argmax, void* stream);

/*
 * One step of the drafter's LSTM cell (Section 3.2.1, Eq. 1-8), for `rows` drafter states at once:
 *   e = E(t)  (Eq. 1, looked up by the caller);   s^m = W^m h + alpha e, m in {f, i, o, c}  (Eq. 2)
 *   g^m = sigmoid(s^m), m in {f, i, o}  (Eq. 5);  s^c = f(s^c) g^i  (Eq. 6);  z = z g^f + s^c  (Eq. 7);
 *   h' = f(z) g^o  (Eq. 8),   f = layer normalisation over the d outputs followed by GeLU.
 * h bf16 [rows, d_in]; emb bf16 [rows, d]; w bf16 [4 d, d_in] = [W^f; W^i; W^o; W^c], each output-major;
 * alpha from owl_lstm_alpha (Eq. 3-4) or the caller; ln_*_gamma / ln_*_beta fp32 [d], the affine parameters of f
 * in Eq. 6 (c) and Eq. 8 (z), NULL for none; eps inside the root of the normalisation (1e-5 customarily);
 * z fp32 [rows, d], read and overwritten (zeros before the first step); h_out_f32 fp32 [rows, d] and
 * h_out_bf16 bf16 [rows, d] receive h' (either may be NULL, not both); workspace fp32 [rows, 4 d], scratch owned
 * by the caller (the call allocates nothing).  The four projections run as one tensor-core product with fp32
 * accumulation, the rest in fp32.  rows <= 384, d_in a multiple of 64, d a multiple of 4 up to 16384.
 * Asynchronous on `stream`; device pointers.
 */
int owl_lstm_cell(owl_ctx* ctx, int32_t rows, int32_t d_in, int32_t d, const void* h, const void* emb,
                  const void* w, float alpha, const float* ln_c_gamma, const float* ln_c_beta,
                  const float* ln_z_gamma, const float* ln_z_beta, float eps, float* z, float* h_out_f32,
                  void* h_out_bf16, float* workspace, void* stream);

/* Eq. 3-4: alpha_0 = 2^(-1/(2 n)), alpha = 2 alpha_0 / ((1 - alpha_0^2) d), n = the tree depth drafted to. */
double owl_lstm_alpha(int32_t n_depth, int32_t d);

/*
 * One whole verify step on device buffers: owl_verify_attn and owl_tree_accept of the same batch
 * (Section 3.2.2 "Decode Stage" followed by the acceptance of the Introduction), arguments as in those
 * two calls, results bit for bit those of the two calls.  The two halves do not depend on each other (the
 * logits are an input), so a small acceptance (total_nodes * ceil(vocab / 8192) <= 1024) costs no launch
 * of its own: spare warps of the attention kernel scan the logits while K/V stream in, and the kernel
 * that merges the attention partials also walks the trees.  Larger scans follow the attention pass as a
 * kernel of their own.  Everything runs on `stream`, in stream order.  Asynchronous; errors as in the
 * two calls (argument errors of either half are reported before anything is launched).
 */
int owl_verify_step(owl_ctx* ctx, const owl_dims* dims, const void* q, const void* k_cache, const void* v_cache,
                    const int32_t* block_table, const int32_t* ctx_lens, const int32_t* node_offsets,
                    const int32_t* tree_parent, void* out, float* lse, const float* logits,
                    const int32_t* draft_tokens, int32_t* accept_len, int32_t* accept_path,
                    int32_t* bonus_token, int32_t* node_argmax, void* stream);

/*
 * One whole verify step from HOST memory: copies every input to device staging buffers owned by
 * the context (grown on demand, so the first call at a given size allocates), runs
 * owl_verify_step, copies the results back and synchronises `stream`.
 * Every tensor pointer here is a HOST pointer (page-locked memory makes the copies asynchronous
 * and fast; pageable memory works).  Shapes and meanings are those of the two calls above;
 * lse_h may be NULL.  Returns a host-detected error, else the device status word (as
 * owl_get_status, which it clears).  Meant for callers without device buffers of their own and
 * for end-to-end timing; a serving loop keeps the KV cache resident and uses the device calls.
 */
int owl_verify_step_host(owl_ctx* ctx, const owl_dims* dims, const void* q_h, const void* k_cache_h,
                         const void* v_cache_h, const int32_t* block_table_h, const int32_t* ctx_lens_h,
                         const int32_t* node_offsets_h, const int32_t* tree_parent_h,
                         const float* logits_h, const int32_t* draft_tokens_h, void* out_h, float* lse_h,
                         int32_t* accept_len_h, int32_t* accept_path_h, int32_t* bonus_token_h,
                         void* stream);

/*
 * Greedy tree acceptance for callers that cannot allocate device memory.  (The paper has no
 * counterpart to this call: it computes exactly what owl_tree_accept computes and exists only
 * because of how some programs manage memory.)
 *
 * Who needs it: an inference server that gave the whole GPU to its own pool at start-up, a
 * plug-in that must stay inside its host's memory budget, or any code on a path where
 * cudaMalloc - and the device-wide synchronisation it can imply - is forbidden.  Such callers
 * cannot use owl_create, which allocates a workspace.  This call takes no context and allocates
 * nothing, neither with cudaMalloc nor through any library: its scratch (one 64-bit arg-max key
 * per logits row and 8192-float vocabulary chunk, a progress counter per sequence, the status word) is a fixed array inside
 * the library image.  The price: every GPU on which the library is loaded holds that array,
 * (OWL_STATIC_MAX_KEYS + 32 + 1024) * 8 bytes = 136.25 KiB, until the process exits.
 *
 * Limit: total_nodes * ceil(vocab / 8192) <= OWL_STATIC_MAX_KEYS (e.g. 1024 nodes at a 128256-entry
 * vocabulary); anything larger returns OWL_ERR_TOO_LARGE and launches nothing.
 *
 * Arguments are those of owl_tree_accept (device pointers, caller-owned), without the context, plus
 * device_status: a device int32 the call first clears and the kernels then set to OWL_ERR_BAD_TREE
 * if a tree is malformed (that sequence's outputs stay unwritten) or node_offsets does not describe
 * total_nodes rows.  With NULL the verdict is dropped: pass a word if malformed input is possible.
 * The work runs on the CURRENT device, on `stream`, asynchronously.
 *
 * Sharing: all calls on a device use the same array.  Calls queued on one stream are safe one after
 * another (a call overwrites every key before it reads it, so stale contents never matter); calls
 * that can overlap on the GPU - different streams, different threads - race on it and must be
 * serialised by the caller.
 *
 * First call: the first call made on each device looks up the array's device address
 * (cudaGetSymbolAddress).  Make that first call outside any stream capture.
 */
#define OWL_STATIC_MAX_KEYS 16384
int owl_tree_accept_static(const owl_dims* dims, const float* logits, const int32_t* draft_tokens,
                           const int32_t* node_offsets, const int32_t* tree_parent, int32_t* accept_len,
                           int32_t* accept_path, int32_t* bonus_token, int32_t* node_argmax,
                           int32_t* device_status, void* stream);

/* Synchronise `stream`, return the device status word of the calls issued on this
 * context since the last owl_get_status (OWL_OK, OWL_ERR_BAD_TREE, OWL_ERR_BAD_PAGE,
 * OWL_ERR_TIMEOUT; the first error wins) and clear it. */
int owl_get_status(owl_ctx* ctx, void* stream);

/*
 * Self-test of the kernels' bounded waits.  Every wait inside the kernels (on a TMA arrival, on a
 * tensor-core commit) gives up after a time limit, raises its CTA's abort flag and reports
 * OWL_ERR_TIMEOUT instead of hanging the GPU.  This call runs that very wait routine in a
 * one-warp kernel on a barrier that nothing ever completes, with the limit given here
 * (1 .. 1e9 ns), then synchronises `stream`.  Returns the device status word and clears it:
 * OWL_ERR_TIMEOUT is the expected answer.  waited_ns (host, may be NULL) receives the nanoseconds
 * the first wait took (about limit_ns) and those of a second wait on the same barrier, which
 * must return at once because the abort flag is up.  Nothing faults or traps; the context stays
 * usable.
 */
int owl_selftest_wait(owl_ctx* ctx, uint64_t limit_ns, uint64_t waited_ns[2], void* stream);

/* Text for a status code; never NULL. */
const char* owl_status_string(int status);

/* Text of the last CUDA error seen by this context ("" if none); valid until the next call. */
const char* owl_last_error(const owl_ctx* ctx);

/* Number of kernels the library has launched through this context since creation. */
int64_t owl_launch_count(const owl_ctx* ctx);

/* Seconds of device time (CUDA events on `stream`) of the most recent call's kernels, by
 * kernel: t[0] verify-attention, t[1] combine, t[2] arg-max with the acceptance walk (one kernel), t[3] = 0.  Only
 * measured while profiling is on (owl_set_profiling(ctx, 1)); synchronises `stream`. */
int owl_set_profiling(owl_ctx* ctx, int on);
int owl_last_kernel_times(owl_ctx* ctx, void* stream, double t[4]);

#ifdef __cplusplus
}
#endif
#endif /* OWLVERIFY_H_ */
