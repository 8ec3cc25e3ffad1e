/*
 * glance.h -- C ABI of the B200 (sm_100a) library for one GLANCE speculative decoding round.
 *
 * The round (Algorithm 1 of the paper; Section 3.1-3.3, Definition 1):
 *   1. glance_draft_block   one pass of the block head -> per-offset top-k ids and log-probabilities
 *   2. glance_build_tree    the N-1 prefixes of highest plug-in score, packed with an ancestor mask
 *   3. glance_verify_tree   one ancestor-masked target pass over the N packed rows
 *   4. glance_accept_commit greedy walk (longest matching prefix) + KV-cache commit/compaction
 *
 * Conventions
 *   - Every function returns an int32 status: GLANCE_OK (0) or a negative GLANCE_E_* code;
 *     glance_status_string() names it.  Argument checks happen on the host before any launch.
 *   - "device" pointers are CUDA device memory owned by the caller and borrowed for the duration
 *     of the context (weights, pools, sequence state) or of the call (inputs and outputs).
 *     "host" pointers are ordinary process memory read during the call only.
 *   - The four round calls, glance_prefill and glance_commit_forced only enqueue work on the
 *     context's stream; they never synchronise and never allocate device memory.  The first call that
 *     meets a buffer it has not seen (a weight matrix, a pool layer, an activation buffer with a new row
 *     count) encodes a TMA descriptor for it on the host and keeps it in the context (a few hundred bytes of
 *     host memory, one driver call, no device work); later calls, CUDA-graph replays included, find it there.
 *   - Faults detected on the device (capacity exceeded, bad index) are recorded in a device status word
 *     read by glance_poll_status(), which synchronises the stream.  The page budget
 *     seq_len + tree_N <= page_size * max_pages_per_seq is one of them (GLANCE_E_CAPACITY): seq_len lives in
 *     device memory, so the host cannot check it before the launch.
 *   - bf16 = raw 16-bit brain-float; all matrices row-major; weights are [out_features, in_features].
 *   - Integer arrays are int32 unless stated.
 */
#ifndef GLANCE_H_
#define GLANCE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    GLANCE_OK = 0,
    GLANCE_E_INVALID_ARG = -1, /* null pointer, negative count, index out of range */
    GLANCE_E_SHAPE = -2,       /* configuration outside the supported shapes */
    GLANCE_E_CAPACITY = -3,    /* workspace or page budget too small */
    GLANCE_E_CUDA = -4,        /* a CUDA runtime call failed */
    GLANCE_E_TIMEOUT = -5,     /* a bounded device-side wait gave up */
    GLANCE_E_BOUNDS = -6,      /* device-side index check failed */
    GLANCE_E_STATE = -7        /* calls out of order (glance_profile_read before glance_profile_enable) */
};

typedef struct glance_ctx glance_ctx;

/* Model and round shape.  Supported: head_dim in {64, 128}; hidden, ffn multiples of 64;
 * 2 <= block_B <= 16; 1 <= topk <= min(16, vocab); 1 <= tree_N <= 128 (tree_N counts the root row: the
 * paper's budget is tree_N - 1, and tree_N = 1 is plain one-token-per-pass decoding through the same calls);
 * page_size = 64; n_q_heads a multiple of n_kv_heads. */
#define GLANCE_MAX_HEAD_LAYERS 8
typedef struct {
    int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
    float rms_eps, rope_theta;
    int32_t block_B, topk, tree_N, page_size, max_batch, max_pages_per_seq;
    /* Block head depth (Section 3.2: five layers whose keys/values are the target's hidden states at five kept
     * layers).  head_layers 0 or 1: one head layer fed by the last target layer (head_taps ignored).  Otherwise
     * head layer i takes its context keys/values from the residual stream after target layer head_taps[i]
     * (0-based, distinct, < n_layers); head_layers <= GLANCE_MAX_HEAD_LAYERS. */
    int32_t head_layers;
    int32_t head_taps[GLANCE_MAX_HEAD_LAYERS];
} glance_config;

/* Target decoder weights (device, bf16).  embed [V,H], lm_head [V,H], final_norm [H].
 * The six per-layer members are HOST arrays of n_layers device pointers:
 * ln1 [H], wqkv [(Hq+2Hkv)d, H] (q rows, then k, then v), wo [H, Hq d], ln2 [H],
 * wgu [2F, H] (gate rows then up rows), wd [H, F]. */
typedef struct {
    const void *embed, *lm_head, *final_norm;
    const void *const *ln1, *const *wqkv, *const *wo, *const *ln2, *const *wgu, *const *wd;
} glance_target_weights;

/* One-layer block head (device, bf16); shares embed and lm_head with the target (Section 3.2).
 * mask_embed [H] fills the masked block slots; ctx_norm [H] normalises the target features that
 * form the head's context keys/values. */
typedef struct {
    const void *ctx_norm, *ln1, *wqkv, *wo, *ln2, *wgu, *wd;
} glance_head_layer;
typedef struct {
    const void *mask_embed, *ctx_norm, *ln1, *wqkv, *wo, *ln2, *wgu, *wd, *final_norm;   /* head layer 0 */
    const glance_head_layer *more;   /* HOST array of head_layers - 1 entries (head layers 1..), or NULL */
} glance_head_weights;

/* Sequence state; every pointer is caller-owned device memory.
 * Cache rows at or beyond seq_len are scratch: the verify pass writes node i at row seq_len + i,
 * so every sequence needs pages covering seq_len + tree_N (and seq_len + block_B for the head).
 * Pool element (layer, page, kv, kv_head, slot, dim) is row-major in that order (kv: 0 = K, 1 = V);
 * logical position p of sequence s lives in page page_table[s][p / page_size], slot p % page_size. */
typedef struct {
    int32_t batch;             /* sequences in this call, <= max_batch */
    int32_t n_pages;           /* pages in each pool (per layer) */
    int32_t *seq_len;          /* [batch] committed length P; updated by commit */
    int32_t *root;             /* [batch] pending root token b; updated by commit */
    const int32_t *page_table; /* [batch][max_pages_per_seq] */
    void *kv_pool;             /* target: [n_layers][n_pages][2][Hkv][page_size][d] bf16 */
    void *head_kv_pool;        /* head:   [head_layers][n_pages][2][Hkv][page_size][d] bf16 */
    void *feat;                /* [head_layers][batch][block_B][H] bf16: tapped target features of the rows
                                  committed last (slice i = the tap of head layer i) */
    int32_t *feat_count;       /* [batch] valid rows in feat (a+1 of the last round, 0 after prefill) */
} glance_seqs;

/* Candidate tree of each sequence (Definition 1), device arrays, N = tree_N rows per sequence.
 * Node 0 is the root; node order is the kept order (score desc, depth asc, path key asc), hence
 * topological.  Rows n_nodes..N-1 are padding (parent -1, visible to themselves only).
 * anc[s][i][w]: bit j of the row (word j>>6, bit j&63) set iff node j is i or an ancestor of i. */
typedef struct {
    int32_t *token, *parent, *depth, *rank; /* [batch][N] */
    float *score;                           /* [batch][N] */
    uint64_t *anc;                          /* [batch][N][(N+63)/64] */
    int32_t *n_nodes;                       /* [batch] */
} glance_tree;

const char *glance_status_string(int32_t status);

/* Bytes of device workspace glance_create needs for this configuration (0 if unsupported). */
size_t glance_workspace_bytes(const glance_config *cfg);

/* Creates a context on the current device.  `workspace` (device, 256-byte aligned, at least
 * glance_workspace_bytes(cfg)) and all weights stay borrowed until glance_destroy.
 * `cuda_stream` is a cudaStream_t (NULL = default stream).  Allocates only host memory; enqueues one small
 * host-to-device copy on that stream (the rotary frequencies theta^(-2i/d), computed in double) and the
 * clearing of the workspace's counters. */
int32_t glance_create(const glance_config *cfg, const glance_target_weights *target,
                      const glance_head_weights *head, void *workspace, size_t workspace_bytes,
                      void *cuda_stream, glance_ctx **out);
int32_t glance_destroy(glance_ctx *ctx);

/* State construction (outside the timed round): causal target forward of `count` new positions of
 * sequence `seq`, appended at seq_len.  Exactly one of `embeds` (device [count,H] bf16: image rows)
 * and `ids` (device [count] int32: text rows) is non-NULL.  Fills target K/V, the head's context
 * K/V, advances seq_len by count, sets root = greedy token after the last row, feat_count = 0. */
int32_t glance_prefill(glance_ctx *ctx, const glance_seqs *seqs, int32_t seq, const void *embeds,
                       const int32_t *ids, int32_t count);

/* Host-side convenience: set seq_len[seq] and root[seq] (rollback; rows beyond are scratch). */
int32_t glance_seq_truncate(glance_ctx *ctx, const glance_seqs *seqs, int32_t seq, int32_t new_len,
                            int32_t new_root);

/* Algorithm 1 line 1 (Section 3.2, Assumption 1).  One pass of the block head: slot 0 = root,
 * slots 1..L masked (L = block_B - 1); every slot attends to all committed context K/V and all
 * block slots.  Also refreshes the head's context K/V for the feat_count rows committed last.
 * Outputs (device): topk_ids [batch][L][k] and topk_lp [batch][L][k] = logit - logsumexp over
 * the full vocabulary, ordered by (logit desc, id asc).  The selection and the log-sum-exp run inside the
 * LM head's epilogue (per 128-feature tile) and one small merge launch; the block's logits are written only on
 * request: logits_dbg (device [batch][block_B][V] fp32) may be NULL. */
int32_t glance_draft_block(glance_ctx *ctx, const glance_seqs *seqs, int32_t *topk_ids, float *topk_lp,
                           float *logits_dbg);

/* Algorithm 1 lines 2-3 (Section 3.3).  Pure function of (root, topk_ids, topk_lp): keeps the
 * min(N-1, sum_l k^l) prefixes of highest score = fl32(score[parent] + lp[depth][rank]) under the
 * order (score desc, depth asc, path key asc) and emits the packed tree with its ancestor mask.
 * `root` is device [batch] (normally seqs->root). */
int32_t glance_build_tree(glance_ctx *ctx, int32_t batch, const int32_t *root, const int32_t *topk_ids,
                          const float *topk_lp, const glance_tree *out);

/* Algorithm 1 line 4 (Definition 1).  Packed target pass: row i = token of node i at position
 * seq_len + depth[i]; attends to all committed positions and to tree rows j with anc[i] bit j;
 * writes K/V of node i at cache row seq_len + i in every layer.
 * Outputs (device): argmax [batch][N] (ties to the lowest id, taken on fp32 accumulators);
 * hidden [head_layers][batch][N][H] bf16: slice i = residual stream after the target layer that head layer i
 * taps (one slice, the stream after the last layer and before the final norm, for the one-layer head);
 * logits_dbg [batch][N][V] fp32 or NULL. */
int32_t glance_verify_tree(glance_ctx *ctx, const glance_seqs *seqs, const glance_tree *tree,
                           int32_t *argmax, void *hidden, float *logits_dbg);

/* Sampling mode (Limitations section: under sampling the walk draws each token from the verified row of its
 * node and descends while the draw is a child).  Same pass as glance_verify_tree, but draws [batch][N] (device)
 * holds one draw per row from softmax(row / temperature) instead of the arg-max; pass it to
 * glance_accept_commit in place of argmax.  The draw is arg-max_v(row[v] / temperature + g(seed, p, v)) where p
 * is the position of the token being drawn (seq_len + depth + 1) and g is standard Gumbel noise
 * -log(-log u), u = ((w >> 9) + 0.5) 2^-23, w = word (v mod 4) of Philox4x32-10 with counter (v / 4, p, 0, 0)
 * and key (seed low word, seed high word): the noise depends on the position, not on the row or the round, so
 * the committed tokens equal plain ancestral sampling with the same field.  temperature > 0 (host value);
 * ties to the lowest id; logits_dbg (if given) receives the unperturbed logits. */
int32_t glance_verify_tree_sample(glance_ctx *ctx, const glance_seqs *seqs, const glance_tree *tree, uint64_t seed,
                                  float temperature, int32_t *draws, void *hidden, float *logits_dbg);

/* Round log for the entropy law (Section 4: the target's next-token entropy H at the round root).  While
 * `entropy` (device, [max_batch] floats) is set, every verify pass -- greedy or sampling -- also writes, for each
 * sequence s, H[s] = -sum_v p_v log p_v in nats with p = softmax of the root row's logits (node 0, temperature 1,
 * no noise), computed from per-tile statistics inside the LM-head epilogue.  NULL switches it off.  Host call. */
int32_t glance_log_root_entropy(glance_ctx *ctx, float *entropy);

/* Algorithm 1 lines 5-12 + commit.  Walks from the root along argmax while the token is a child
 * in the tree; then, per layer, moves cache row seq_len + path[d] to row seq_len + d (d = 1..a),
 * gathers hidden[path[0..a]] into feat (every tap slice), sets feat_count = a+1, seq_len += a+1, root = new root.
 * Outputs (device): accept_len [batch] = a; path [batch][block_B] node indices (path[0] = 0);
 * out_tokens [batch][block_B]: the a accepted tokens followed by the new root. */
int32_t glance_accept_commit(glance_ctx *ctx, const glance_seqs *seqs, const glance_tree *tree,
                             const int32_t *argmax, const void *hidden, int32_t *accept_len, int32_t *path,
                             int32_t *out_tokens);

/* Test hook (teacher forcing): commit a caller-given path instead of walking.
 * path [batch][block_B] (device), path_len [batch] = a+1 (device), new_root [batch] (device). */
int32_t glance_commit_forced(glance_ctx *ctx, const glance_seqs *seqs, const void *hidden,
                             const int32_t *path, const int32_t *path_len, const int32_t *new_root);

/* Synchronises the stream and returns the device status word (GLANCE_OK or the first fault);
 * the word is cleared. */
int32_t glance_poll_status(glance_ctx *ctx, int32_t *device_status);

/* Test hook: the attention kernel alone.  q (device [batch*T][Hq*d] bf16) attends, per sequence, to cache
 * rows 0..seq_len-1 of target layer `layer` (all visible) and to rows seq_len..seq_len+T-1 under
 * anc (device [batch][T][(T+63)/64], or NULL = all visible); out (device [batch*T][Hq*d] bf16).
 * q_lo and out_lo (same layouts, either may be NULL) are the second bf16 terms of the queries and of the
 * outputs: the value is hi + lo, as between the kernels of a pass.
 * This is the masked attention of Definition 1's packed pass in isolation. */
int32_t glance_debug_attention(glance_ctx *ctx, const glance_seqs *seqs, int32_t layer, const void *q,
                               const void *q_lo, const uint64_t *anc, int32_t T, void *out, void *out_lo);

/* Test hook / tuning knob: second bf16 terms of the attention on key tiles that lie entirely inside the committed
 * context (tiles holding tree or block keys always keep both terms).  lo_skip bit 0: such a tile's score MMAs use the
 * queries' first term only; bit 1: its P V MMAs use the probabilities' first term only; applied to sequences with at
 * least min_keys committed positions.  Host call; takes effect from the next enqueued pass (a captured CUDA graph
 * keeps the setting it was captured with). */
int32_t glance_debug_attention_terms(glance_ctx *ctx, int32_t lo_skip, int32_t min_keys);

/* Test hook: the weight-streaming GEMM kernel alone (K % 64 == 0).  mode 0: Y[s][r][f] fp32 planes (S splits);
 * mode 1: W = [2F][K] (gate rows then up rows), act (device [R][F] bf16) = silu(gate) * up;
 * mode 2: argmax (device [R] int32) over f of X W^T with ties to the lowest f, Y (device [R][Nout] fp32) optional. */
int32_t glance_debug_gemm(glance_ctx *ctx, int32_t mode, const void *W, const void *X, float *Y, void *act,
                             int32_t *argmax, int32_t Nout, int32_t K, int32_t R, int32_t S);

/* Test hook for the bounded device waits (every mbarrier wait of the tcgen05 kernels gives up after a limit, records
 * GLANCE_E_TIMEOUT in the status word, lets the CTA drain the copies it has in flight, free its tensor memory and
 * return).  One shot: in the NEXT glance_debug_gemm launch the TMA producer never fills the ring slot of k-step
 * `kstep` (0-based, of every CTA's own K range) and every wait of that launch gives up after wait_limit_ns
 * (1 us .. 1 s) instead of the regular second, so the MMA issuer's wait on that slot runs out.  Nothing faults and
 * nothing is left in flight; the launch's results are undefined, the status word reads GLANCE_E_TIMEOUT, and the
 * context stays usable. */
int32_t glance_debug_stall_next_gemm(glance_ctx *ctx, int32_t kstep, uint64_t wait_limit_ns);

/* Test hook: phase timestamps of the GEMM kernel.  While a buffer (device, slots x 16 uint64) is set, the
 * n-th GEMM launch after this call makes its first CTA write nanosecond timestamps (entry, set-up done,
 * predecessor finished, first tile landed, accumulator ready, cluster barrier 1, tile shipped, cluster
 * barrier 2, epilogue done, exit) into entries 0-11 of slot n % slots (attention launches count too and record
 * their own phases).  Entries 12-15 are merged over ALL CTAs of the launch with atomic max / min, so the caller
 * presets them (12, 15 to 0; 13, 14 to all ones): 12 = last main loop end, 13 = first main loop end, 14 = first
 * CTA start, 15 = last CTA end.  buffer = NULL, slots = 0 switches it off. */
int32_t glance_debug_trace(glance_ctx *ctx, uint64_t *buffer, int32_t slots);

/* Measurement aid.  While enabled, every kernel launch is bracketed by a pair of CUDA events on the context's
 * stream (the pairs are created when profiling is first enabled, so the round calls still allocate nothing).
 * glance_profile_read synchronises the stream and fills three arrays of GLANCE_PROFILE_KINDS entries, indexed by
 * kernel kind (0 weight-streaming GEMM, 1 attention, 2 row setup, 3 top-k / tree / walk+commit, 4 everything
 * else): summed device time in milliseconds, summed algorithmic bytes (GEMM only: weights once +
 * activations in + results out) and launch count; then it resets the tally.  Disabling only pauses the
 * tally.  At most 32768 launches are tallied per read.  glance_profile_read on a context where profiling was
 * never enabled returns GLANCE_E_STATE. */
#define GLANCE_PROFILE_KINDS 5
int32_t glance_profile_enable(glance_ctx *ctx, int32_t on);
int32_t glance_profile_read(glance_ctx *ctx, double *ms, double *bytes, int64_t *launches);

/* Per-offset top-k and log-softmax without any caller-provided workspace.  (The paper has no counterpart:
 * this entry point exists for callers that cannot allocate device memory -- a process whose GPU memory was
 * handed to its own arena at start-up, a plug-in inside a host framework's callback, a loop that cannot
 * afford the device-wide synchronisation an allocation may trigger.)
 * Same computation as the last step of glance_draft_block: for each sequence s and offset j = 1..L of
 * logits (device [batch][block_B][vocab] fp32, row 0 of each sequence ignored) the k largest entries ordered
 * by (logit desc, id asc) and lp = logit - logsumexp over the whole vocabulary, into topk_ids / topk_lp
 * (device [batch][L][k]).  Work is enqueued on `cuda_stream`; nothing is allocated or freed.
 * Scratch lives in a 1 MiB device array inside the library (held by every GPU that loads it, until exit);
 * a call needing more -- batch*(block_B-1)*ceil(vocab/1024)*(8k+8) bytes, rounded up to 256 for the first
 * part -- returns GLANCE_E_CAPACITY and launches nothing.  The first call on each device looks up the
 * array's device address (with that device current); make that first call before starting any stream
 * capture.  All calls share the one array: calls that may overlap on the GPU (different streams, no
 * ordering between them) race on it and must be serialised by the caller. */
int32_t glance_topk_static(const float *logits, int32_t batch, int32_t block_B, int32_t vocab, int32_t k,
                           int32_t *topk_ids, float *topk_lp, void *cuda_stream);

/* Number of kernel launches enqueued by this context since creation (host counter). */
int64_t glance_launch_count(const glance_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* GLANCE_H_ */
