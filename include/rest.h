/*
 * rest.h - C ABI of the GPU hot path of one REST decoding step
 * (Retrieval-Based Speculative Decoding, arXiv 2311.08252).
 *
 * Set-up:       rest_suffix_array_build (_full, _in_groups, _append), rest_datastore_create
 *               (Sec. 3.2, datastore construction)
 * Draft side:   rest_draft                                 (Sec. 3.2, Algorithms 1 and 2)
 *               rest_retrieve, rest_gather_rows, rest_draft_from_runs: the same in pieces, for a
 *               datastore spread over several GPUs
 * Verify side:  rest_tree_attention, rest_accept           (Sec. 3.2, draft verification / acceptance)
 * Between steps: rest_kv_commit                            (the accepted path joins the prefix)
 * Health:       rest_device_error_flags
 * (measurement and planning aids live in rest_aids.h)
 *
 * Conventions
 *   - Every pointer named d_* is a DEVICE pointer owned by the caller.  The library borrows
 *     it for the duration of the call (the datastore handle: for its lifetime), never frees
 *     it and never allocates device memory.  Scratch space is passed in by the caller; its
 *     size comes from the matching *_workspace_bytes query.
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and return
 *     without synchronising (rest_datastore_create with REST_DS_VALIDATE is the exception).
 *   - Host-checkable problems return a non-zero rest_status before anything is launched.
 *     Data-dependent problems are reported per context in d_status and give an empty tree.
 *     Nothing aborts, traps or throws.
 *   - All integer outputs are fully determined by the inputs (no dependence on scheduling).
 */
#ifndef REST_H_
#define REST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t rest_status;
enum {
  REST_OK = 0,
  REST_INVALID_ARG = 1,         /* null pointer, negative size, inconsistent shapes          */
  REST_UNSUPPORTED = 2,         /* outside the limits listed at rest_draft / rest_tree_attention */
  REST_WORKSPACE_TOO_SMALL = 3,
  REST_CUDA_ERROR = 4,          /* a CUDA runtime call failed; see rest_last_cuda_error()    */
  REST_BAD_DATASTORE = 5        /* validation found an unsorted / non-permutation suffix array
                                   or a token outside [0, vocab)                              */
};

/* Per-context codes written to d_status by rest_draft. */
enum {
  REST_CTX_OK = 0,
  REST_CTX_BAD_TOKEN = 1,       /* one of the last n_max context tokens is outside [0, vocab) */
  REST_CTX_BAD_DATASTORE = 2,   /* suffix-array entry out of range, or gathered continuations
                                   not in lexicographic order                                 */
  REST_CTX_INTERNAL = 3
};

enum { REST_SAMPLE_STRIDED = 0, REST_SAMPLE_FIRST_K = 1 };
/* How rest_draft searches the suffix array (rest_draft_params.search_path); the results are the
 * same either way.  SINGLE: every suffix length at once, a warp per length, 32 probes per round
 * inside the range that the datastore's n-gram index gives for the query's first tokens (fewest
 * dependent reads, the fastest single context); 512 or 1024 threads per context.  BATCHED: 256
 * threads per context, six or seven searches instead of fifteen (the lengths that match are
 * n_min ... n* without a gap) and eight probes per round once the probes leave L2: more
 * dependent rounds, fewer random DRAM reads, more contexts in flight (most of all with the
 * scratch that rest_draft_workspace_bytes asks for, see d_ws).  AUTO picks BATCHED when the call
 * has at least 5 contexts per SM and that scratch, or at least 16 contexts per SM without it. */
enum { REST_SEARCH_AUTO = 0, REST_SEARCH_SINGLE = 1, REST_SEARCH_BATCHED = 2 };
enum { REST_DS_VALIDATE = 1u, REST_DS_INDEX = 2u };

/* Limits of this implementation. */
enum {
  REST_MAX_SUFFIX = 16,   /* n_max */
  REST_MAX_M = 16,        /* continuation length */
  REST_MAX_N = 256,       /* draft tokens per tree */
  REST_MAX_K = 32768,     /* candidates per context */
  REST_HEAD_DIM = 128
};

typedef struct rest_datastore rest_datastore;   /* opaque host object holding device pointers */

/* Draft hyper-parameters (Sec. 4.1 "Hyperparameters": n_max = 16, m = 10, c = 64).
 *   n_max, n_min  longest / shortest context suffix tried by Algorithm 1 (1 <= n_min <= n_max <= 16)
 *   K             cap on the number of continuation candidates used per context (1..32768)
 *   m             continuation length (1..16)
 *   N             maximum number of draft tokens, the paper's c (1..256)
 *   sample_mode   which K of cnt > K matches are used: REST_SAMPLE_STRIDED takes suffix-array
 *                 slot lo + floor(j*cnt/K), REST_SAMPLE_FIRST_K takes lo + j, j = 0..K-1
 *   search_path   REST_SEARCH_AUTO / SINGLE / BATCHED: a performance switch, never a result */
typedef struct {
  int32_t n_max, n_min, K, m, N, sample_mode, search_path;
} rest_draft_params;

/*
 * Datastore (Sec. 3.2 "Datastore construction" and "Retrieving from the datastore": a token
 * stream whose every position is a (context, continuation) pair, indexed by a suffix array).
 *
 *   d_tokens   int32[n_tokens], values in [0, vocab), vocab < 2^31
 *   d_sa       int32[n_tokens] (sa_bytes = 4, n_tokens < 2^31) or int64[n_tokens] (sa_bytes = 8):
 *              start positions of all suffixes in lexicographic order of their tokens (compared
 *              as unsigned integers, a suffix that is a proper prefix of another sorts first).
 *              Only the order on the first n_max + m tokens matters to rest_draft.
 *   flags      REST_DS_VALIDATE: check on the device that d_sa is a permutation ordered on the
 *              first 32 tokens and that tokens are in range; synchronises `stream`; returns
 *              REST_BAD_DATASTORE on failure.
 *              REST_DS_INDEX: build a bucket index into d_aux (asynchronously on `stream`): for
 *              every token the suffix-array range of the suffixes that start with it, and a hash
 *              table with the ranges of the frequent sequences of two, three and four tokens
 *              (up to 512 MiB).  rest_draft then starts each search inside such a range instead
 *              of over the whole array, and a frequent suffix of up to four tokens needs no
 *              search at all: fewer dependent reads, identical results.  Needs vocab <= 2^22
 *              (ignored beyond).
 *   d_aux      device scratch of rest_datastore_aux_bytes() bytes, 256-byte aligned, needed with
 *              either flag (NULL otherwise).  With REST_DS_INDEX the handle keeps using it: it
 *              must stay allocated and untouched until rest_datastore_destroy.
 *   out        receives a host handle; free it with rest_datastore_destroy (device arrays stay
 *              the caller's).
 */
size_t rest_datastore_aux_bytes(uint64_t n_tokens, int32_t sa_bytes, uint32_t vocab);
rest_status rest_datastore_create(const int32_t* d_tokens, uint64_t n_tokens, const void* d_sa,
                                  int32_t sa_bytes, uint32_t vocab, uint32_t flags, void* d_aux,
                                  size_t aux_bytes, void* stream, rest_datastore** out);
void rest_datastore_destroy(rest_datastore* ds);

/*
 * rest_datastore_create_shard - a datastore whose suffix array lists only n_sa <= n_tokens of
 * the positions, e.g. one shard of a token stream that is spread over several GPUs (Sec. 5,
 * "Effect of the datastore size": the datastore may outgrow one device).  A shard holds the
 * tokens of its own position range followed by the first tokens of the next shard (at least
 * n_max + m of them), and its suffix array orders the positions of its own range only, so that
 * every occurrence in the whole stream is found by exactly one shard and its continuation is
 * complete.  Everything else as rest_datastore_create; d_sa has n_sa entries, all distinct
 * positions in [0, n_tokens), ordered like a suffix array.
 */
rest_status rest_datastore_create_shard(const int32_t* d_tokens, uint64_t n_tokens, const void* d_sa,
                                        uint64_t n_sa, int32_t sa_bytes, uint32_t vocab, uint32_t flags,
                                        void* d_aux, size_t aux_bytes, void* stream, rest_datastore** out);

/*
 * rest_draft - Algorithm 1 (longest-suffix exact-match retrieval), Algorithm 2 (Trie weights,
 * the c heaviest nodes) and the breadth-first pseudo sequence with its tree-attention mask
 * (Sec. 3.2 "Draft verification"), for B independent contexts.
 *
 * Per context b:
 *   1. n runs from min(n_max, ctx_len[b]) down to n_min; q = last n context tokens; [lo, hi) is
 *      the suffix-array range of suffixes starting with q; the first non-empty range wins.
 *      No match (or ctx_len < n_min): empty tree, match_n = 0.  That is not an error.
 *   2. Candidates: the min(hi-lo, K) sampled slots (see sample_mode); candidate j is the up to m
 *      tokens that follow the match, cut at the end of the token stream.
 *   3. Trie node = distinct non-empty prefix of a candidate; weight = number of candidates
 *      having that prefix.  Kept: the N largest by (weight desc, depth asc, token path asc).
 *   4. Output order: by depth, then token path (breadth first, siblings ascending by token).
 *
 *   d_ctx        int32, context b starts at d_ctx + b*ctx_stride and holds ctx_len[b] tokens
 *   d_tokens     int32[B,N]  draft tokens;           unused slots -1
 *   d_parents    int32[B,N]  index of the parent node, -1 for children of the root; unused -1
 *   d_depth      int32[B,N]  1-based depth;          unused 0
 *   d_pos_ids    int32[B,N]  ctx_len + depth - 1;    unused ctx_len
 *   d_mask       uint32[B,N,ceil(N/32)]  bit (j & 31) of word (j >> 5) of row i is set iff node
 *                j is node i or an ancestor of i; unused rows hold their own bit only
 *   d_n_nodes    int32[B]
 *   d_match_n    int32[B]    matched suffix length (0 = none)
 *   d_match_range int64[B,2] lo, hi of the matched suffix-array range
 *   d_node_count int32[B,N]  weight of each kept node (may be NULL)
 *   d_status     int32[B]    REST_CTX_* code
 *   d_ws         optional scratch of rest_draft_workspace_bytes() bytes, 16-byte aligned (the
 *                query answers for the current device and may be 0).  Never needed for the
 *                results, only for speed; with NULL or fewer bytes every path runs as one launch
 *                of one block per context.  What it buys:
 *                - single-context path, 2 to 1024 contexts (48 to 1024 when K < 8192; never when
 *                  K <= 512): a context with a long candidate list lets idle blocks (those of
 *                  finished or lighter contexts, and blocks started on SMs that have no context)
 *                  read part of its rows; the scratch holds the contexts' counters and
 *                  node-start bitmaps (about 6 m K / 32 bytes per context).  The call zeroes the
 *                  counters itself.
 *                - batched path: three launches (search; build of the contexts with few
 *                  candidates on small blocks; build of the others on large blocks); the scratch
 *                  holds the two context lists (8 bytes per context).
 *                The scratch must not be shared by calls that may run at the same time.
 */
size_t rest_draft_workspace_bytes(const rest_draft_params* params, int32_t B);
rest_status rest_draft(const rest_datastore* ds, const rest_draft_params* params,
                       const int32_t* d_ctx, int64_t ctx_stride, const int32_t* d_ctx_len,
                       int32_t B, int32_t* d_tokens, int32_t* d_parents, int32_t* d_depth,
                       int32_t* d_pos_ids, uint32_t* d_mask, int32_t* d_n_nodes,
                       int32_t* d_match_n, int64_t* d_match_range, int32_t* d_node_count,
                       int32_t* d_status, void* d_ws, size_t ws_bytes, void* stream);

/*
 * The draft in pieces, for a datastore spread over several GPUs (Algorithms 1 and 2 over the
 * union of the shards; Sec. 5 "Effect of the datastore size").  Per decoding step:
 *   1. every GPU:  rest_retrieve on its shard -> its longest matching suffix length and range;
 *   2. exchange:   the winning length n* is the maximum over the shards (a shorter suffix of a
 *                  match is a match, so a shard either matches n* or contributes nothing);
 *                  shards that match n* report their hit counts cnt_i; with cnt = sum cnt_i,
 *                  shard i contributes all its rows when cnt <= K, else
 *                  floor(K C_i / cnt) - floor(K C_(i-1) / cnt) rows (C_i = cnt_1 + ... + cnt_i),
 *                  spread over its range like rest_draft spreads K over one range.  With one
 *                  shard this is exactly rest_draft's rule;
 *   3. every GPU:  rest_gather_rows -> its rows, in lexicographic order (one sorted run);
 *   4. exchange:   the runs of all shards travel to the GPU that builds the tree;
 *   5. builder:    rest_draft_from_runs merges the runs and runs Algorithm 2 and the tree
 *                  emission unchanged.
 * The exchanges are ordinary collectives on small tensors and belong to the caller (the Python
 * package does them with torch.distributed).
 *
 * rest_retrieve       Algorithm 1 alone: d_match_n[b], d_match_range[b] = {lo, hi}, d_status[b];
 *                     arguments as in rest_draft (K, m, N, sample_mode of `params` are not used).
 * rest_gather_rows    candidate j < take[b] of context b: the suffix-array slot
 *                     lo + floor(j cnt / take[b]) (lo + j with REST_SAMPLE_FIRST_K or when
 *                     take[b] = cnt), its up to m tokens after the match into d_rows[b][j][0..m)
 *                     (zero padded) and their number into d_row_len[b][j]; rows j >= take[b] get
 *                     length 0.  d_match_n / d_match_range as written by rest_retrieve (a shard
 *                     that lost sets take[b] = 0).  Kr = row capacity per context (<= 32768).
 *                     d_status[b] is OR-ed with REST_CTX_BAD_DATASTORE on an entry out of range.
 * rest_draft_from_runs  d_rows int32[B][R][Kr][m], d_row_len int32[B][R][Kr], d_run_rows
 *                     int32[B][R] (rows of run r in use; each run in lexicographic order, a row
 *                     that is a prefix of another first; R * Kr <= 32768).  Outputs as rest_draft
 *                     (d_node_count may be NULL); runs out of order give status
 *                     REST_CTX_BAD_DATASTORE and an empty tree.  d_ws: scratch of
 *                     rest_draft_from_runs_workspace_bytes(B, R, Kr) bytes.
 */
rest_status rest_retrieve(const rest_datastore* ds, const rest_draft_params* params,
                          const int32_t* d_ctx, int64_t ctx_stride, const int32_t* d_ctx_len,
                          int32_t B, int32_t* d_match_n, int64_t* d_match_range, int32_t* d_status,
                          void* stream);
rest_status rest_gather_rows(const rest_datastore* ds, const rest_draft_params* params,
                             const int32_t* d_match_n, const int64_t* d_match_range,
                             const int32_t* d_take, int32_t B, int32_t Kr, int32_t* d_rows,
                             int32_t* d_row_len, int32_t* d_status, void* stream);
size_t rest_draft_from_runs_workspace_bytes(int32_t B, int32_t R, int32_t Kr);
rest_status rest_draft_from_runs(const rest_draft_params* params, const int32_t* d_rows,
                                 const int32_t* d_row_len, const int32_t* d_run_rows, int32_t R,
                                 int32_t Kr, const int32_t* d_ctx_len, int32_t B, int32_t* d_tokens,
                                 int32_t* d_parents, int32_t* d_depth, int32_t* d_pos_ids,
                                 uint32_t* d_mask, int32_t* d_n_nodes, int32_t* d_node_count,
                                 int32_t* d_status, void* d_ws, size_t ws_bytes, void* stream);

/*
 * rest_tree_attention - attention of the N draft positions of each context over the prefix
 * KV cache and over their own ancestors (Sec. 3.2 "Draft verification": the pseudo sequence
 * is run with an attention mask under which every token sees exactly its dependencies).
 *
 *   For context b, head h, node i:  keys = {0..L-1} U {L+j : bit j of mask row i}, L = kv_len[b];
 *   out = softmax(scale * q.k) v  with natural exponent, fp32 accumulation, bf16 output.
 *
 *   d_q       bf16, element (b,i,h,d) at b*strides[0] + i*strides[1] + h*strides[2] + d
 *   d_k, d_v  bf16, element (b,hk,l,d) at b*strides[3] + hk*strides[4] + l*strides[5] + d;
 *             rows L..L+N-1 hold the K/V of the draft nodes; hk = h / (H / H_kv)
 *   d_out     bf16, element (b,i,h,d) at b*strides[6] + i*strides[7] + h*strides[8] + d
 *   strides   host array of 9 element strides; rows of D elements are contiguous and every
 *             stride is a multiple of 8 elements (16-byte rows); base pointers 16-byte aligned
 *   d_kv_len  int32[B], 0 <= L and L + N <= rows available
 *   max_kv    upper bound on L + N over the batch (sizes the split of the key range)
 *   d_mask    uint32[B,N,ceil(N/32)] as written by rest_draft
 *   d_lse     optional float[B,H,N]: log of the softmax denominator (natural log, of scaled
 *             scores); with N > 64 the denominator sums the bf16-rounded probabilities that the
 *             output is built from, so it carries bf16 precision (a few 1e-3 absolute)
 *   d_ws      scratch of rest_tree_attention_workspace_bytes() bytes
 *   scale     softmax scale, finite and > 0 (else REST_INVALID_ARG)
 *   Limits: D = 128; 1 <= N <= 256 (any tree rest_draft can write); H % H_kv == 0.
 */
size_t rest_tree_attention_workspace_bytes(int32_t B, int32_t H, int32_t N, int32_t D,
                                           int32_t max_kv);
rest_status rest_tree_attention(const void* d_q, const void* d_k, const void* d_v,
                                const int64_t* strides, const int32_t* d_kv_len,
                                const uint32_t* d_mask, int32_t B, int32_t H, int32_t H_kv,
                                int32_t N, int32_t D, int32_t max_kv, float scale, void* d_out,
                                float* d_lse, void* d_ws, size_t ws_bytes, void* stream);

/*
 * rest_tree_attention_static_scratch - rest_tree_attention for callers that cannot allocate.
 *
 * (The paper has no counterpart; this is a packaging variant of the call above.)
 *
 * Some users of this library cannot obtain the workspace that rest_tree_attention asks for:
 * a serving process that handed every free byte of device memory to its own KV-cache pool at
 * start-up, or a decode loop whose rules forbid allocation calls because cudaMalloc/cudaFree
 * may stall the whole device.  For them the split-KV partials live in a fixed array of
 * REST_STATIC_SCRATCH_BYTES (768 KiB) inside the library image.  Every GPU that loads the
 * library holds that array until the process exits, whether or not this call is used.
 *
 *   - Arguments, layouts, results and limits are those of rest_tree_attention, without
 *     d_ws / ws_bytes.  The call itself performs no device or host allocation.
 *   - Returns REST_WORKSPACE_TOO_SMALL, launching nothing, when
 *     rest_tree_attention_workspace_bytes(B, H, N, D, max_kv) exceeds REST_STATIC_SCRATCH_BYTES.
 *     Scratch is only needed when one (context, head) pair is cut into more than 8 key ranges,
 *     i.e. for very few pairs with long caches, and then holds one partial of N x 130 floats per
 *     cluster of 8 ranges; no more clusters are used than the GPU can run at once (about 30).
 *     B*H = 2, N = 64, max_kv = 4160 needs 0.51 MiB and fits; B*H = 1, N = 64, max_kv = 16448
 *     needs about 1 MiB and is refused.
 *   - The first call on each device looks up the array's device address (one runtime query,
 *     with that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left.
 *     That is harmless here: each call writes every partial it later reads, so nothing has to
 *     start at zero.  But two calls whose kernels may overlap on the GPU (different streams)
 *     race on the array: serialise them.
 */
enum { REST_STATIC_SCRATCH_BYTES = 768 * 1024 };
rest_status rest_tree_attention_static_scratch(
    const void* d_q, const void* d_k, const void* d_v, const int64_t* strides,
    const int32_t* d_kv_len, const uint32_t* d_mask, int32_t B, int32_t H, int32_t H_kv, int32_t N,
    int32_t D, int32_t max_kv, float scale, void* d_out, float* d_lse, void* stream);

/*
 * rest_accept - draft acceptance (Sec. 3.2 "Draft acceptance": draft tokens are accepted from
 * the start while they coincide with the tokens sampled from the verifier; everything after
 * the first mismatch is rejected).
 *
 *   d_verifier_tokens int32[B,N+1]: slot 0 = verifier's token after the prefix, slot i+1 = its
 *                     token after draft node i (greedy argmax or a sampled token).
 *   Walk from the root: if the current node has a child whose token equals the verifier's token
 *   at the current node, accept it and continue from that child; stop otherwise or after
 *   max_depth accepted nodes.
 *   d_accept_len   int32[B]
 *   d_accept_nodes int32[B,max_depth]    accepted node indices, unused -1
 *   d_out_tokens   int32[B,max_depth+1]  accepted tokens followed by the verifier's token at the
 *                  stopping node (what plain decoding would emit next); unused -1
 */
rest_status rest_accept(const int32_t* d_tokens, const int32_t* d_parents,
                        const int32_t* d_n_nodes, const int32_t* d_verifier_tokens, int32_t B,
                        int32_t N, int32_t max_depth, int32_t* d_accept_len,
                        int32_t* d_accept_nodes, int32_t* d_out_tokens, void* stream);

/*
 * rest_kv_commit - make the accepted draft path part of the prefix KV cache.
 *
 * The paper does not describe the cache; any implementation of its loop (Sec. 3.2: draft,
 * verify, accept, repeat with the longer context) has to do this between two steps.  For
 * context b with L = kv_len[b] and len = accept_len[b]: K/V row L + accept_nodes[b][i] of every
 * kv head is copied to row L + i, i = 0..len-1, in place (accept_nodes[b][i] >= i always holds
 * for trees written by rest_draft, and the kernel reads all source rows before it writes).
 *
 *   d_k, d_v        bf16, element (b,hk,l,d) at b*kv_strides[0] + hk*kv_strides[1] + l*kv_strides[2] + d,
 *                   same layout rules as rest_tree_attention (D = 128, 16-byte aligned rows)
 *   d_accept_nodes  int32[B,max_depth], d_accept_len int32[B]: as written by rest_accept
 *   N               number of tree slots (node indices are clamped to [0, N))
 *   d_new_kv_len    optional int32[B]: receives L + len (may alias d_kv_len)
 *   Limits: max_depth <= 16.  The token the verifier produced at the stop (out_tokens[len]) has
 *   no K/V yet: it is the next step's first input token.
 */
rest_status rest_kv_commit(void* d_k, void* d_v, const int64_t* kv_strides, const int32_t* d_kv_len,
                           const int32_t* d_accept_nodes, const int32_t* d_accept_len, int32_t B,
                           int32_t H_kv, int32_t N, int32_t D, int32_t max_depth,
                           int32_t* d_new_kv_len, void* stream);

/*
 * rest_suffix_array_build - the datastore's suffix array, built on the device (Sec. 3.2
 * "Datastore construction"; "Retrieving from the datastore" matches through a suffix array).
 * Set-up work: call it once, then rest_datastore_create on the result.
 *
 *   Order: suffixes compare on their first 32 tokens (unsigned, a suffix that ends early is
 *   smaller); suffixes equal on those are ordered by position.  rest_draft reads at most
 *   n_max + m <= 32 tokens of a suffix, so its results are those of the full order.
 *
 *   d_tokens  int32[n_tokens] device, values in [0, 2^31 - 1)
 *   sa_bytes  4 or 8: d_sa is int32[n_tokens] (n_tokens < 2^31) or int64[n_tokens] (device, written)
 *   d_ws      device scratch, 256-byte aligned.  Two methods, picked by what fits:
 *             - up to 2^31 - 1 tokens and at least rest_suffix_array_workspace_bytes(n_tokens)
 *               (about 32 bytes per token + 64 MiB): prefix doubling, five sorts of the whole
 *               stream, asynchronous on `stream`;
 *             - otherwise (longer streams, or a smaller workspace): positions are put into
 *               buckets by first token and groups of whole buckets are sorted one after the
 *               other on their packed 32-token keys.  Scratch: 32 bytes per position of the
 *               largest group + 0.2 GiB; rest_suffix_array_workspace_bytes answers for groups of
 *               2^30 positions, rest_suffix_array_min_workspace_bytes for groups just large
 *               enough for the most frequent first token.  This method reads the bucket
 *               histogram back (it synchronises `stream`) and returns REST_UNSUPPORTED when one
 *               first token starts more suffixes than the workspace can sort at once.
 *   Limits: n_tokens <= 2^40.
 */
size_t rest_suffix_array_workspace_bytes(uint64_t n_tokens);
size_t rest_suffix_array_min_workspace_bytes(uint64_t n_tokens, uint64_t largest_bucket);
rest_status rest_suffix_array_build(const int32_t* d_tokens, uint64_t n_tokens, int32_t sa_bytes,
                                    void* d_sa, void* d_ws, size_t ws_bytes, void* stream);
/* The true suffix array (whole suffixes compared, no ties left): prefix doubling carried on
 * past 32 tokens until every suffix is distinct, one flag read back per extra round (the call
 * synchronises `stream`).  Streams of up to 2^31 - 1 tokens; workspace as for the first method.
 * rest_draft gives the same results on either array; this one is for callers who want the
 * array itself. */
rest_status rest_suffix_array_build_full(const int32_t* d_tokens, uint64_t n_tokens, int32_t sa_bytes,
                                         void* d_sa, void* d_ws, size_t ws_bytes, void* stream);
/*
 * rest_suffix_array_append - the suffix array after n_new tokens were appended to a stream of
 * n_old tokens (Sec. 3.2 "Datastore construction": a datastore that grows).  Only the suffixes
 * of the last 31 old positions and of the new tokens can change place under the 32-token
 * order; they are sorted by themselves and merged into the old array in one pass.
 *   d_tokens   int32[n_old + n_new]: the whole stream, old tokens first
 *   d_sa_old   the array of the first n_old tokens as rest_suffix_array_build wrote it (NULL when n_old = 0)
 *   d_sa_new   receives n_old + n_new entries of sa_bytes bytes; must not be d_sa_old
 *   d_ws       rest_suffix_array_append_workspace_bytes(n_new) bytes (about 44 bytes per new
 *              token + 64 MiB), 256-byte aligned.  Asynchronous on `stream`.
 */
size_t rest_suffix_array_append_workspace_bytes(uint64_t n_new);
rest_status rest_suffix_array_append(const int32_t* d_tokens, uint64_t n_old, uint64_t n_new,
                                     const void* d_sa_old, int32_t sa_bytes, void* d_sa_new,
                                     void* d_ws, size_t ws_bytes, void* stream);
/* The second method whatever the size: groups of at most max_group positions (0: as many as the
 * workspace allows; at least the count of the most frequent first token). */
rest_status rest_suffix_array_build_in_groups(const int32_t* d_tokens, uint64_t n_tokens,
                                              int32_t sa_bytes, void* d_sa, uint64_t max_group,
                                              void* d_ws, size_t ws_bytes, void* stream);

/*
 * Device-side trouble that no per-call status can carry.  Every wait inside the kernels is
 * bounded; a kernel that gives up sets a bit here instead of spinning, and its output is then
 * undefined.  Reads and clears the flags of the current device (synchronises the device).
 *   bit 0: tree attention gave up waiting for its tensor-core work
 *   bit 1: tree attention found its shared-memory window misaligned and did nothing
 */
rest_status rest_device_error_flags(uint32_t* h_flags);

const char* rest_status_string(rest_status s);
/* Text of the last CUDA runtime error seen by this library on the calling thread. */
const char* rest_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* REST_H_ */
