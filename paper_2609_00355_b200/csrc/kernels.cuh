// Launch wrappers of the round's kernels (definitions in the .cu files beside this header).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace glance {

// ---- setup (kernels_small.cu) -------------------------------------------------------------
// what a setup kernel emits per row besides the bookkeeping: fp32 residual x, bf16 x * gain, sum of squares
struct RowOut {
    int H;
    float *x;            // [R][H]
    bf16 *xb;            // [R][H] first term of bf16(x * gain)
    bf16 *xb_lo;         // [R][H] second term (x * gain - first term), or nullptr
    float *ssq;          // [n_ssq][ssq_stride]: plane 0 gets the row's full sum of squares, the others 0
    int n_ssq, ssq_stride;
};

struct VerifySetup {
    // rows r = s*N + i
    int batch, N, d;
    float theta;
    const int32_t *seq_len;     // [batch]
    const int32_t *token;       // [batch][N] tree tokens (mode tree) or nullptr
    const int32_t *depth;       // [batch][N] (mode tree) or nullptr (chain: depth = i)
    const bf16 *row_embeds;     // prefill: [count][H] or nullptr
    const int32_t *row_ids;     // prefill: [count] or nullptr
    int count;                  // prefill: valid rows
    uint64_t *chain_anc;        // prefill: [N][W] written with the causal chain mask
    const bf16 *embed;          // [V][H]
    const bf16 *gain;           // first norm's gain
    int vocab;
    int capacity;               // max_pages_per_seq * page
    KvGeom geom;
    const int32_t *page_table;  // [batch][max_pages_per_seq]
    RowOut out;
    RowMeta meta;
    int32_t *status;
};
void launch_setup_verify(const VerifySetup &p, cudaStream_t st);

struct DraftSetup {
    // block rows r = s*B + j (R1 = batch*n_block rows), then feature rows r = R1 + s*FR + i
    int batch, B, FR, d;
    float theta;
    const int32_t *seq_len, *root;
    const bf16 *feat;           // [batch][FR][H]: FR = B (round) or tree_N (prefill head-context update)
    const int32_t *feat_count;  // [batch] or nullptr (then count_const rows, appended at seq_len)
    int count_const;
    int n_block;                // B (round) or 0 (prefill: only feature rows)
    int features_only;          // 1: leave the block rows alone (head layers 1..: their inputs come from the layer below)
    const bf16 *embed, *mask_embed;
    const bf16 *gain_block, *gain_feat;   // head input norm / context norm
    int vocab;
    int capacity;
    KvGeom geom;
    const int32_t *page_table;
    RowOut out;
    RowMeta meta;
    int32_t *status;
};
void launch_setup_draft(const DraftSetup &p, cudaStream_t st);

// rows (s, j), j = 1..L of logits [batch*B][V] -> ids/lp [batch][L][k]; scratch: cand [rows][topk_warps(V)][k],
// ml [rows][topk_warps(V)][2].  Two launches.
int topk_warps(int V);
void launch_topk(const float *logits, int batch, int B, int V, int k, int32_t *ids, float *lp,
                 unsigned long long *cand, float *ml, cudaStream_t st);

// merge of the draft LM head's per-tile candidates and log-sum-exp shares (gemm_tc_kernel mode 5): thr [batch*B][16],
// ml [tiles][batch*B][2], cnt [tiles][batch*B], cand [tiles][batch*B][kTopkTileCap] -> ids / lp [batch][B-1][k];
// re-arms thr.  One launch.
void launch_topk_merge(int batch, int B, int tiles, int k, uint32_t *thr, const float *ml, const int32_t *cnt,
                       const unsigned long long *cand, int32_t *ids, float *lp, cudaStream_t st);

// ---- tree + walk (tree_walk.cu) -----------------------------------------------------------
void launch_build_tree(int batch, int N, int L, int k, const int32_t *root, const int32_t *ids, const float *lp,
                       const glance_tree &out, cudaStream_t st);

struct WalkCommit {
    int batch, N, B, H, n_layers;
    const int32_t *token, *parent, *n_nodes;   // tree (walk mode) or nullptr
    const int32_t *argmax;                      // [batch][N] (walk mode)
    const int32_t *forced_path, *forced_len, *forced_root;   // forced mode (argmax == nullptr)
    const bf16 *hidden;                         // [n_taps][batch][N][H]
    int n_taps;                                 // head layers = tapped target layers
    bf16 *kv_pool;
    KvGeom geom;
    const int32_t *page_table;
    int32_t *seq_len, *root, *feat_count;
    bf16 *feat;                                 // [n_taps][batch][B][H]
    int32_t *accept_len, *path, *out_tokens;    // outputs (may be nullptr in forced mode)
    int32_t *counters;                          // [batch], zero between calls
    int32_t *status;
};
void launch_walk_commit(const WalkCommit &p, cudaStream_t st);

// prefill bookkeeping: seq_len += count, root = argmax[count-1], feat_count = 0
void launch_prefill_advance(int32_t *seq_len, int32_t *root, int32_t *feat_count, const int32_t *argmax, int count,
                            cudaStream_t st);

// ---- attention (attention_tc.cu) ----------------------------------------------------------
struct AttnParams {
    int batch, T, Hq, Hkv, d;    // T = query rows per sequence = extra (uncommitted) keys per sequence
    const bf16 *q;               // [batch*T][Hq*d]
    const bf16 *q_lo;            // second term of the two-term queries (same layout), or nullptr
    const bf16 *pool_layer;
    KvGeom geom;
    const int32_t *page_table;
    const int32_t *seq_len;
    const uint64_t *anc;         // [batch][T][W] or nullptr (all T extra keys visible)
    int W;
    bf16 *out;                   // [batch*T][Hq*d]
    bf16 *out_lo;                // second term of the two-term output, or nullptr
    int S;                       // key splits (= cluster size)
    // Second bf16 terms on key tiles that lie entirely inside the committed context: bit 0 set = the score MMAs of
    // such a tile use the queries' first term only, bit 1 set = its P V MMAs use the probabilities' first term only.
    // Applied to sequences with at least lo_skip_min_keys committed positions (tiles that hold tree / block keys
    // always keep both terms).
    int lo_skip, lo_skip_min_keys;
    int32_t *status;
    unsigned long long *trace;   // test hook: phase timestamps of the first CTA, or nullptr
};
// map_kv = 2-D map of the pool layer {d, n_pages*2*Hkv*64 rows}, box {64, 64}
cudaError_t launch_attention_tc(const AttnParams &p, const CUtensorMap &map_kv, cudaStream_t st);
int attention_tc_q_tiles(int T, int G);
int attention_tc_splits(int T, int G, int Hkv, int batch, int d);

}  // namespace glance
