/*
 * CPU oracle for the verify step of long-context speculative decoding
 * (tree-masked attention of drafted tokens against a KV cache + greedy acceptance).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * step computes; it shares no code with the CUDA library and the product path
 * never calls it.  Only the tests, the smoke check and the benchmark's
 * CPU-baseline leg load it.
 *
 * What it follows in the paper:
 *  - "Decode Stage" paragraph (Section 3.2.2): the drafted tree is verified in one
 *    pass in which every node (including an appended [SPEC] leaf) attends to the
 *    context plus exactly the nodes on its own root path - the worked example lists
 *    the paths (t_{N+1}), (t_{N+1}, t_{N+2}), (t_{N+1}, t_{N+2'}).
 *  - Introduction / Related Work: the target model verifies all drafted tokens in
 *    parallel and the decoding algorithm accepts the tokens that keep the output
 *    distribution; "acceptance length" (caption of Figure 1) is the number of
 *    tokens accepted per verification step.  Under greedy decoding a drafted token
 *    keeps the distribution iff it equals the target's own arg-max continuation of
 *    its parent.
 *  - Non-tree verification (Section 3.2.3, NonTreeVerify of Algorithm 1) is the same pass with
 *    a chain-shaped tree.
 *  - Around that pass (Algorithm 1): Prepare(d) appends the [SPEC] leaves and fixes mask and
 *    position ids; the accepted path names the [SPEC] whose hidden state the drafter gets; the
 *    accepted tokens are then committed to the cache ("l <- l; d").
 *
 * Parity pins (tests, CPU only): brute-force dense-mask softmax in numpy fp64,
 * single-node == decode attention and chain == causal attention against a library
 * SDPA in fp64, the paper's worked mask example, softmax invariants, hand-worked
 * acceptance cases, losslessness on a toy model, a closed-form expectation, and
 * the acceptance-length bounds the paper states; for the steps around the pass the
 * paper's [SPEC] example extended to leaf indices and position ids, hand-worked
 * commits on shuffled page tables, the same commit on a gathered logical view, and
 * the multi-step lossless loop with the cache contents checked.  No function here is unpinned.
 *
 * Arithmetic: bf16 inputs are decoded exactly to double; dot products, the
 * two-pass softmax and the weighted sum run in double; nothing is blocked, fused
 * or reordered.  Outputs are double (not rounded to bf16).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_BAD_ARG (-1)
#define ORACLE_BAD_TREE (-2)
#define ORACLE_BAD_PAGE (-3)

int owl_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static double bf16_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* IEEE binary16 to double, by the format's definition: sign, 5 exponent bits (bias 15), 10 fraction bits;
 * exponent 0 = subnormal (fraction * 2^-24), exponent 31 = infinity or NaN. */
static double f16_to_double(uint16_t h) {
    const int sign = h >> 15, e = (h >> 10) & 31, f = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)f, -24);
    else if (e == 31) v = f ? NAN : INFINITY;
    else v = ldexp((double)(1024 + f), e - 25);
    return sign ? -v : v;
}

/* Element type of q / k_cache / v_cache: 0 = bf16 (the benchmark configurations), 1 = fp16 (the paper's own
 * precision, Appendix "Inference Details"). */
static double elem_to_double(uint16_t h, int is_f16) { return is_f16 ? f16_to_double(h) : bf16_to_double(h); }

/* Sequence that owns packed node `n` (node_offsets has B+1 entries). */
static int seq_of_node(const int32_t* node_offsets, int B, int n) {
    for (int b = 0; b < B; ++b)
        if (n >= node_offsets[b] && n < node_offsets[b + 1]) return b;
    return -1;
}

/* Pointer to the D values of token `pos` of sequence b, KV head h, in the paged cache
 * laid out [page][kv_head][slot][d]. */
static const uint16_t* kv_row(const uint16_t* cache, const int32_t* block_table, int b,
                              int max_pages_per_seq, int num_pages, int Hkv, int page_size, int D,
                              int h, int64_t pos) {
    int64_t lp = pos / page_size, slot = pos % page_size;
    int32_t page = block_table[(int64_t)b * max_pages_per_seq + lp];
    if (page < 0 || page >= num_pages) return NULL;
    return cache + (((int64_t)page * Hkv + h) * page_size + slot) * D;
}

/* Check the node order the interface requires: node 0 is the only root, parent[i] < i. */
static int tree_ok(const int32_t* parent, int n) {
    if (n < 1 || parent[0] != -1) return 0;
    for (int i = 1; i < n; ++i)
        if (parent[i] < 0 || parent[i] >= i) return 0;
    return 1;
}

/*
 * Tree-masked attention, one (packed node, query head) row at a time.
 *
 * Row (n, hq): let b be the sequence of node n, i its local index, L = ctx_lens[b].
 * Visible keys = {0..L-1} (the whole committed context) plus L+j for every j on the
 * root path of i, found by following parent pointers from i (i itself included).
 *   s_k = sm_scale * <q, K_k>;  m = max s_k;  Z = sum exp(s_k - m)
 *   lse = m + ln Z;  out = sum exp(s_k - m) V_k / Z
 *
 * rows: if row_node == NULL every (n, hq) pair is computed in order n*Hq + hq and
 * n_rows must be N*Hq; otherwise rows r = (row_node[r], row_head[r]).
 * out is [n_rows, D] doubles, lse [n_rows] doubles.
 */
static int attn_any(int is_f16, int B, int Hq, int Hkv, int D, int page_size, int max_pages_per_seq,
                    int num_pages, double sm_scale, const uint16_t* q, const uint16_t* k_cache,
                    const uint16_t* v_cache, const int32_t* block_table, const int32_t* ctx_lens,
                    const int32_t* node_offsets, const int32_t* tree_parent, int64_t n_rows,
                    const int32_t* row_node, const int32_t* row_head, double* out, double* lse) {
    if (B < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || D < 1 || page_size < 1) return ORACLE_BAD_ARG;
    const int G = Hq / Hkv;
    const int N = node_offsets[B];
    if (row_node == NULL && n_rows != (int64_t)N * Hq) return ORACLE_BAD_ARG;
    for (int b = 0; b < B; ++b)
        if (!tree_ok(tree_parent + node_offsets[b], node_offsets[b + 1] - node_offsets[b]))
            return ORACLE_BAD_TREE;

    int status = ORACLE_OK;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        const int n = row_node ? row_node[r] : (int)(r / Hq);
        const int hq = row_head ? row_head[r] : (int)(r % Hq);
        const int b = seq_of_node(node_offsets, B, n);
        if (b < 0 || hq < 0 || hq >= Hq) {
#pragma omp atomic write
            status = ORACLE_BAD_ARG;
            continue;
        }
        const int base = node_offsets[b];
        const int nb = node_offsets[b + 1] - base;
        const int i = n - base;
        const int64_t L = ctx_lens[b];
        const int h = hq / G;
        const int32_t* parent = tree_parent + base;

        /* visible keys: prefix, then the root path of i by literal pointer chasing */
        int64_t nvis = 0;
        int64_t* vis = (int64_t*)malloc((size_t)(L + nb) * sizeof(int64_t));
        double* s = (double*)malloc((size_t)(L + nb) * sizeof(double));
        for (int64_t k = 0; k < L; ++k) vis[nvis++] = k;
        {
            char* on_path = (char*)calloc((size_t)nb, 1);
            for (int j = i; j >= 0; j = parent[j]) on_path[j] = 1;
            for (int j = 0; j < nb; ++j)
                if (on_path[j]) vis[nvis++] = L + j;
            free(on_path);
        }

        const uint16_t* qrow = q + ((int64_t)n * Hq + hq) * D;
        int bad = 0;
        double m = -INFINITY;
        for (int64_t t = 0; t < nvis; ++t) {
            const uint16_t* krow = kv_row(k_cache, block_table, b, max_pages_per_seq, num_pages,
                                          Hkv, page_size, D, h, vis[t]);
            if (!krow) { bad = 1; break; }
            double acc = 0.0;
            for (int d = 0; d < D; ++d) acc += elem_to_double(qrow[d], is_f16) * elem_to_double(krow[d], is_f16);
            s[t] = sm_scale * acc;
            if (s[t] > m) m = s[t];
        }
        if (bad) {
#pragma omp atomic write
            status = ORACLE_BAD_PAGE;
            free(vis); free(s);
            continue;
        }
        double Z = 0.0;
        for (int64_t t = 0; t < nvis; ++t) Z += exp(s[t] - m);
        double* o = out + r * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        for (int64_t t = 0; t < nvis; ++t) {
            const uint16_t* vrow = kv_row(v_cache, block_table, b, max_pages_per_seq, num_pages,
                                          Hkv, page_size, D, h, vis[t]);
            const double p = exp(s[t] - m);
            for (int d = 0; d < D; ++d) o[d] += p * elem_to_double(vrow[d], is_f16);
        }
        for (int d = 0; d < D; ++d) o[d] /= Z;
        lse[r] = m + log(Z);
        free(vis); free(s);
    }
    return status;
}

int owl_oracle_attn(int B, int Hq, int Hkv, int D, int page_size, int max_pages_per_seq,
                    int num_pages, double sm_scale, const uint16_t* q, const uint16_t* k_cache,
                    const uint16_t* v_cache, const int32_t* block_table, const int32_t* ctx_lens,
                    const int32_t* node_offsets, const int32_t* tree_parent, int64_t n_rows,
                    const int32_t* row_node, const int32_t* row_head, double* out, double* lse) {
    return attn_any(0, B, Hq, Hkv, D, page_size, max_pages_per_seq, num_pages, sm_scale, q, k_cache, v_cache, block_table,
                    ctx_lens, node_offsets, tree_parent, n_rows, row_node, row_head, out, lse);
}

/* The same attention with q, k_cache and v_cache in fp16, the data type the paper ran in (Appendix "Inference Details"). */
int owl_oracle_attn_f16(int B, int Hq, int Hkv, int D, int page_size, int max_pages_per_seq,
                        int num_pages, double sm_scale, const uint16_t* q, const uint16_t* k_cache,
                        const uint16_t* v_cache, const int32_t* block_table, const int32_t* ctx_lens,
                        const int32_t* node_offsets, const int32_t* tree_parent, int64_t n_rows,
                        const int32_t* row_node, const int32_t* row_head, double* out, double* lse) {
    return attn_any(1, B, Hq, Hkv, D, page_size, max_pages_per_seq, num_pages, sm_scale, q, k_cache, v_cache, block_table,
                    ctx_lens, node_offsets, tree_parent, n_rows, row_node, row_head, out, lse);
}

/* Decoders exposed for their own pin (every bit pattern against a library conversion). */
void owl_oracle_decode16(const uint16_t* in, int64_t count, int is_f16, double* out) {
    for (int64_t i = 0; i < count; ++i) out[i] = elem_to_double(in[i], is_f16);
}

/*
 * Row arg-max over the vocabulary: the smallest index attaining the row maximum.
 * Scalar scan with a strict '>' so the first maximum wins; NaN is read as -inf
 * (so +0.0 and -0.0 tie and an all-NaN row gives 0).
 */
void owl_oracle_argmax(const float* logits, int64_t N, int64_t V, int32_t* am) {
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        const float* row = logits + n * V;
        float best = isnan(row[0]) ? -INFINITY : row[0];
        int32_t bi = 0;
        for (int64_t j = 1; j < V; ++j) {
            float x = isnan(row[j]) ? -INFINITY : row[j];
            if (x > best) { best = x; bi = (int32_t)j; }
        }
        am[n] = bi;
    }
}

/*
 * Greedy tree acceptance.  The root is the target's own, already chosen token and
 * is always accepted.  A non-root node c is accepted iff every edge (p -> c') on
 * its root path has a drafted token draft[c'] >= 0 equal to am[p], the target's
 * arg-max continuation of p.  The winner is the accepted node of greatest depth
 * (lowest index among equals); accept_len = depth + 1 (nodes on the path, root
 * included), accept_path lists the path root -> winner padded with -1, and
 * bonus_token = am[winner] is the target's next token after the accepted path.
 */
int owl_oracle_accept(int B, const int32_t* node_offsets, const int32_t* tree_parent,
                      const int32_t* draft_tokens, const int32_t* am, int path_stride,
                      int32_t* accept_len, int32_t* accept_path, int32_t* bonus_token) {
    for (int b = 0; b < B; ++b) {
        const int base = node_offsets[b];
        const int nb = node_offsets[b + 1] - base;
        const int32_t* parent = tree_parent + base;
        if (!tree_ok(parent, nb)) return ORACLE_BAD_TREE;
        int win = 0, win_depth = 0;
        for (int i = 0; i < nb; ++i) {
            int ok = 1, depth = 0;
            for (int c = i; parent[c] >= 0; c = parent[c]) {
                const int p = parent[c];
                if (!(draft_tokens[base + c] >= 0 && draft_tokens[base + c] == am[base + p])) ok = 0;
                ++depth;
            }
            if (ok && depth > win_depth) { win = i; win_depth = depth; }
        }
        if (win_depth + 1 > path_stride) return ORACLE_BAD_ARG;
        accept_len[b] = win_depth + 1;
        for (int k = 0; k < path_stride; ++k) accept_path[(int64_t)b * path_stride + k] = -1;
        int k = win_depth;
        for (int c = win; c >= 0; c = parent[c]) accept_path[(int64_t)b * path_stride + k--] = c;
        bonus_token[b] = am[base + win];
    }
    return ORACLE_OK;
}

/*
 * Prepare(d) of Algorithm 1 / Section 3.2.2 "Decode Stage": one [SPEC] token is appended after every
 * tree path, i.e. every drafted node j (the end of the path root..j) gets one [SPEC] child, "the same
 * number of [SPEC] as the number of tree nodes", in node order (the paper's example: the first [SPEC]
 * follows (t_{N+1}), the second (t_{N+1}, t_{N+2}), the third (t_{N+1}, t_{N+2'})).  The attention mask
 * follows from the parent array; the manipulated position id of a token is the number of context tokens
 * plus its depth in the tree (a token on a path sits where it would sit if that path were the text).
 *
 * In: B trees (node_offsets, tree_parent, draft_tokens; the root's token is t_{N+1}), ctx_lens,
 * the token id of [SPEC].  Out, for sequence b with n nodes, 2n nodes at out_offsets[b] = 2 * node_offsets[b]:
 *   nodes 0..n-1   the drafted tree as given; nodes n..2n-1 the [SPEC] leaves, leaf n + j child of j
 *   out_draft      drafted token, -1 for a [SPEC] leaf (never a candidate of the acceptance)
 *   out_input_ids  what the verifier embeds: drafted token, spec_token for a leaf
 *   out_position   ctx_lens[b] + depth
 */
int owl_oracle_prepare_spec(int B, const int32_t* node_offsets, const int32_t* tree_parent,
                            const int32_t* draft_tokens, const int32_t* ctx_lens, int32_t spec_token,
                            int32_t* out_offsets, int32_t* out_parent, int32_t* out_draft,
                            int32_t* out_input_ids, int32_t* out_position) {
    out_offsets[0] = 0;
    for (int b = 0; b < B; ++b) {
        const int base = node_offsets[b], n = node_offsets[b + 1] - base;
        const int32_t* parent = tree_parent + base;
        if (!tree_ok(parent, n)) return ORACLE_BAD_TREE;
        const int ob = 2 * base;
        out_offsets[b + 1] = ob + 2 * n;
        for (int j = 0; j < n; ++j) {
            int depth = 0;
            for (int c = j; parent[c] >= 0; c = parent[c]) ++depth;
            out_parent[ob + j] = parent[j];
            out_draft[ob + j] = draft_tokens[base + j];
            out_input_ids[ob + j] = draft_tokens[base + j];
            out_position[ob + j] = ctx_lens[b] + depth;
            out_parent[ob + n + j] = j;                 /* the [SPEC] after the path that ends in j */
            out_draft[ob + n + j] = -1;
            out_input_ids[ob + n + j] = spec_token;
            out_position[ob + n + j] = ctx_lens[b] + depth + 1;
        }
    }
    return ORACLE_OK;
}

/*
 * "When a path is accepted, we take the hidden state of the corresponding [SPEC]" (Section 3.2.2, Decode
 * Stage): the [SPEC] leaf (a child with a negative draft token) of the last node of the accepted path;
 * the lowest index if there were several, -1 if the node has none (a tree verified without [SPEC]).
 */
int owl_oracle_spec_leaf(int B, const int32_t* node_offsets, const int32_t* tree_parent,
                         const int32_t* draft_tokens, const int32_t* accept_len, const int32_t* accept_path,
                         int path_stride, int32_t* spec_node) {
    for (int b = 0; b < B; ++b) {
        const int base = node_offsets[b], n = node_offsets[b + 1] - base;
        if (accept_len[b] < 1 || accept_len[b] > path_stride) return ORACLE_BAD_ARG;
        const int last = accept_path[(int64_t)b * path_stride + accept_len[b] - 1];
        if (last < 0 || last >= n) return ORACLE_BAD_ARG;
        spec_node[b] = -1;
        for (int c = n - 1; c >= 0; --c)
            if (tree_parent[base + c] == last && draft_tokens[base + c] < 0) spec_node[b] = c;
    }
    return ORACLE_OK;
}

/*
 * Commit of the accepted tokens to the cache: Algorithm 1, "l <- l; d" and "N <- N + |d|".  During the
 * verification the K/V of drafted node i sit at logical position L + i.  After it the accepted path
 * p_0 = 0 < p_1 < ... < p_{a-1} becomes text: the token at L + p_k moves to L + k for every KV head, K and
 * V alike, everything else that was drafted is dropped, and the committed length grows by a.
 * All rows are read before any is written (a position may be both a source and a destination).
 */
int owl_oracle_kv_commit(int B, int Hkv, int D, int page_size, int max_pages_per_seq, int num_pages,
                         uint16_t* k_cache, uint16_t* v_cache, const int32_t* block_table, int32_t* ctx_lens,
                         const int32_t* node_offsets, const int32_t* accept_len, const int32_t* accept_path,
                         int path_stride) {
    for (int b = 0; b < B; ++b) {
        const int n = node_offsets[b + 1] - node_offsets[b];
        const int a = accept_len[b];
        const int32_t* path = accept_path + (int64_t)b * path_stride;
        if (a < 1 || a > n || a > path_stride || path[0] != 0) return ORACLE_BAD_ARG;
        for (int k = 1; k < a; ++k)
            if (path[k] <= path[k - 1] || path[k] >= n) return ORACLE_BAD_ARG;
        const int64_t L = ctx_lens[b];
        uint16_t* tmp = (uint16_t*)malloc((size_t)2 * a * Hkv * D * sizeof(uint16_t));
        for (int k = 0; k < a; ++k)
            for (int h = 0; h < Hkv; ++h) {
                const uint16_t* ks = kv_row(k_cache, block_table, b, max_pages_per_seq, num_pages, Hkv, page_size, D, h, L + path[k]);
                const uint16_t* vs = kv_row(v_cache, block_table, b, max_pages_per_seq, num_pages, Hkv, page_size, D, h, L + path[k]);
                if (!ks || !vs) { free(tmp); return ORACLE_BAD_PAGE; }
                memcpy(tmp + ((size_t)(2 * k) * Hkv + h) * D, ks, (size_t)D * sizeof(uint16_t));
                memcpy(tmp + ((size_t)(2 * k + 1) * Hkv + h) * D, vs, (size_t)D * sizeof(uint16_t));
            }
        for (int k = 0; k < a; ++k)
            for (int h = 0; h < Hkv; ++h) {
                uint16_t* kd = (uint16_t*)kv_row(k_cache, block_table, b, max_pages_per_seq, num_pages, Hkv, page_size, D, h, L + k);
                uint16_t* vd = (uint16_t*)kv_row(v_cache, block_table, b, max_pages_per_seq, num_pages, Hkv, page_size, D, h, L + k);
                if (!kd || !vd) { free(tmp); return ORACLE_BAD_PAGE; }
                memcpy(kd, tmp + ((size_t)(2 * k) * Hkv + h) * D, (size_t)D * sizeof(uint16_t));
                memcpy(vd, tmp + ((size_t)(2 * k + 1) * Hkv + h) * D, (size_t)D * sizeof(uint16_t));
            }
        free(tmp);
        ctx_lens[b] = (int32_t)(L + a);
    }
    return ORACLE_OK;
}

/*
 * The routing of Algorithm 1 (Section 3.2.3), one decision per sequence and step.  `score` is the non-tree
 * drafter's estimate of its acceptance length, c the threshold (the paper sets c = 9, the longest acceptance
 * the tree drafter can reach, Appendix "Inference Details").
 *   score > c            -> non-tree verification of the chain as drafted, no [SPEC]; lastwaslinear <- true
 *   else, lastwaslinear  -> tree from the drafter trained WITHOUT [SPEC] (the last step produced no [SPEC]
 *                           hidden state); lastwaslinear <- false
 *   else                 -> tree from the drafter trained WITH [SPEC]
 * Either tree is verified with [SPEC] leaves appended.  route: 0 = linear, 1 = tree / D_nospec, 2 = tree / D_spec.
 */
void owl_oracle_howl_route(int B, const float* score, float c, uint8_t* lastwaslinear, int32_t* route) {
    for (int b = 0; b < B; ++b) {
        if (score[b] > c) {
            lastwaslinear[b] = 1;
            route[b] = 0;
        } else if (lastwaslinear[b]) {
            route[b] = 1;
            lastwaslinear[b] = 0;
        } else {
            route[b] = 2;
        }
    }
}

/*
 * Prepare(d) on a routed batch: a sequence routed to non-tree verification (route 0) keeps its chain as drafted
 * ("we do not append any [SPEC] to the input in this case", Section 3.2.3); every other sequence gets one [SPEC]
 * leaf per node as in owl_oracle_prepare_spec.  Outputs are packed sequence after sequence (n or 2n nodes).
 */
int owl_oracle_prepare_hybrid(int B, const int32_t* node_offsets, const int32_t* tree_parent,
                              const int32_t* draft_tokens, const int32_t* ctx_lens, const int32_t* route,
                              int32_t spec_token, int32_t* out_offsets, int32_t* out_parent, int32_t* out_draft,
                              int32_t* out_input_ids, int32_t* out_position) {
    out_offsets[0] = 0;
    for (int b = 0; b < B; ++b) {
        const int base = node_offsets[b], n = node_offsets[b + 1] - base;
        const int32_t* parent = tree_parent + base;
        if (!tree_ok(parent, n)) return ORACLE_BAD_TREE;
        const int ob = out_offsets[b];
        const int with_spec = route[b] != 0;
        out_offsets[b + 1] = ob + (with_spec ? 2 * n : n);
        for (int j = 0; j < n; ++j) {
            int depth = 0;
            for (int c = j; parent[c] >= 0; c = parent[c]) ++depth;
            out_parent[ob + j] = parent[j];
            out_draft[ob + j] = draft_tokens[base + j];
            out_input_ids[ob + j] = draft_tokens[base + j];
            out_position[ob + j] = ctx_lens[b] + depth;
            if (with_spec) {
                out_parent[ob + n + j] = j;
                out_draft[ob + n + j] = -1;
                out_input_ids[ob + n + j] = spec_token;
                out_position[ob + n + j] = ctx_lens[b] + depth + 1;
            }
        }
    }
    return ORACLE_OK;
}
