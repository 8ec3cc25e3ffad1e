// C ABI of the GLANCE round library: context, workspace carving, and the stream-ordered sequence of
// kernels behind each entry point declared in glance.h.
#include <algorithm>
#include <cmath>
#include <map>
#include <new>
#include <tuple>
#include <vector>

#include "gemm_tc.cuh"
#include "kernels.cuh"

using namespace glance;

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// split-K factor of a weight-streaming GEMM: as many CTAs as fit one wave at two CTAs per SM (one CTA per SM
// keeps too few weight bytes in flight to cover the HBM latency), at least 7 k-tiles per split
// The splits of one tile form a thread-block cluster (<= 8 CTAs) that reduces them through shared memory.
// With more than one 128-row block the launch is tensor-bound, not latency-bound: every (tile, row block) item is a
// long main loop, and splitting K only pays where it evens out the last wave over the 148 SMs -- each split adds a
// cluster epilogue of a few microseconds per item.
int choose_split(int Nout, int K, int rows, bool two_term) {
    const int tiles = (Nout + 127) / 128;
    const int ktiles = K / 64;
    const int row_blocks = (rows + 127) / 128;
    if (row_blocks > 1) {
        // Two CTAs per SM keep about 200 KB of operands in flight, which is what the tensor rate needs from L2; one
        // CTA per SM runs at about half of it.  So a wave is 296 items wide, each item running at half an SM's rate.
        const double step_us = two_term ? 0.45 : 0.225;       // one 128 x 128-row x 64 k-step at an SM's tensor rate
        const double unit_us = ktiles * step_us;               // one unsplit item with the SM to itself
        const int smax = std::max(1, std::min(8, ktiles / 7));
        int best = 1;
        double best_us = 1e30;
        for (int s = 1; s <= smax; ++s) {
            const double waves = std::ceil((double)tiles * row_blocks * s / 296.0);
            // cluster epilogue per wave; clusters of a later wave also wait for enough SMs of one GPC to come free together
            const double epilogue_us = s == 1 ? 0.0 : (waves > 1.0 ? 10.0 : 3.0);
            const double us = waves * (2.0 * unit_us / s + epilogue_us);
            if (us < best_us - 1e-9) { best_us = us; best = s; }
        }
        return best;
    }
    int s = (2 * 148) / tiles;
    s = std::min(s, std::max(1, ktiles / 7));
    s = std::max(1, std::min(s, 8));
    if (s == 8 && tiles > 33) s = 7;                   // at most 33 clusters of eight are resident at two CTAs per SM
    return s;
}

struct Workspace {
    float *x;            // [Rmax][H] residual stream
    bf16 *xn;            // [2][Rmax][H] bf16(x * gain) as two terms (hi plane, lo plane); so are attn and act
    bf16 *q;             // [Rmax][Hq d]
    bf16 *attn;          // [Rmax][Hq d]
    bf16 *act;           // [Rmax][F]
    int32_t *walk_ctr;
    int32_t *row_seq, *row_pos;
    long long *row_kvrow;
    float *ssq;            // [n_ssq][Rmax] per-tile sums of squares of the residual rows
    float *rope_cos, *rope_sin;
    double *inv_freq;      // [d/2]
    uint64_t *chain_anc;   // [N][W] prefill chain mask
    bf16 *hidden_tmp;      // [head layers][N][H] prefill: tapped hidden states of the chunk
    int32_t *argmax_tmp;   // [N]
    int32_t *status;
    unsigned long long *am_keys;   // [Rlog] packed arg-max keys, zero between launches
    int32_t *am_counter;
    float *ent_part;       // [vocab tiles][max_batch][3] soft-max statistics of the root rows (entropy log)
    // draft top-k, fused into the LM head: per 128-feature tile and block row
    uint32_t *tk_thr;              // [batch*B][kTopkTileCap] running class maxima of every row (0 between launches)
    float *tk_ml;                  // [vocab tiles][batch*B][2] (max, sum exp)
    int32_t *tk_cnt;               // [vocab tiles][batch*B] candidate keys emitted
    unsigned long long *tk_cand;   // [vocab tiles][batch*B][kTopkTileCap]
    size_t total;
};

struct Dims {
    int Rmax, Rlog, qkv_out, qd, W, n_ssq;
};

Dims make_dims(const glance_config &c) {
    Dims d;
    d.Rmax = c.max_batch * std::max(c.tree_N, 2 * c.block_B);
    d.Rmax = std::max(d.Rmax, c.tree_N);
    d.Rlog = c.max_batch * std::max(c.tree_N, c.block_B);
    d.qkv_out = (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
    d.qd = c.n_q_heads * c.head_dim;
    d.n_ssq = (c.hidden + 127) / 128;
    d.W = (c.tree_N + 63) / 64;
    return d;
}

// carve (or just size, when base == nullptr) the workspace
Workspace carve(const glance_config &c, const Dims &d, unsigned char *base) {
    Workspace w;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        unsigned char *p = base ? base + off : nullptr;
        off = align_up(off + bytes, 256);
        return p;
    };
    const size_t R = d.Rmax, H = c.hidden;
    w.x = (float *)take(R * H * 4);
    w.xn = (bf16 *)take(2 * R * H * 2);                 // two planes: hi, lo
    w.q = (bf16 *)take(2 * R * d.qd * 2);               // two planes
    w.attn = (bf16 *)take(2 * R * d.qd * 2);            // two planes
    w.act = (bf16 *)take(2 * R * (size_t)c.ffn * 2);    // two planes
    w.walk_ctr = (int32_t *)take((size_t)c.max_batch * 4);
    w.row_seq = (int32_t *)take(R * 4);
    w.row_pos = (int32_t *)take(R * 4);
    w.row_kvrow = (long long *)take(R * 8);
    w.ssq = (float *)take((size_t)d.n_ssq * R * 4);
    w.rope_cos = (float *)take(R * (c.head_dim / 2) * 4);
    w.rope_sin = (float *)take(R * (c.head_dim / 2) * 4);
    w.inv_freq = (double *)take((size_t)(c.head_dim / 2) * 8);
    w.chain_anc = (uint64_t *)take((size_t)c.tree_N * d.W * 8);
    w.hidden_tmp = (bf16 *)take((size_t)(c.head_layers > 1 ? c.head_layers : 1) * c.tree_N * H * 2);
    w.argmax_tmp = (int32_t *)take((size_t)c.tree_N * 4);
    w.status = (int32_t *)take(256);
    w.am_keys = (unsigned long long *)take((size_t)d.Rlog * 8);
    w.am_counter = (int32_t *)take(256);
    w.ent_part = (float *)take((size_t)((c.vocab + 127) / 128) * c.max_batch * 3 * 4);
    const size_t trows = (size_t)((c.vocab + 127) / 128) * c.max_batch * c.block_B;
    w.tk_thr = (uint32_t *)take((size_t)c.max_batch * c.block_B * kTopkTileCap * 4);
    w.tk_ml = (float *)take(trows * 2 * 4);
    w.tk_cnt = (int32_t *)take(trows * 4);
    w.tk_cand = (unsigned long long *)take(trows * kTopkTileCap * 8);
    w.total = off;
    return w;
}

bool config_ok(const glance_config *c) {
    if (!c) return false;
    if (c->n_layers < 1 || c->hidden < 64 || c->hidden % 64 || c->ffn < 64 || c->ffn % 64) return false;
    if (c->head_dim != 64 && c->head_dim != 128) return false;
    if (c->n_q_heads < 1 || c->n_kv_heads < 1 || c->n_q_heads % c->n_kv_heads) return false;
    if (c->vocab < 2) return false;
    if (c->block_B < 2 || c->block_B > kMaxBlock || c->topk < 1 || c->topk > kMaxTopk || c->topk > c->vocab) return false;
    if (c->tree_N < 1 || c->tree_N > kMaxTreeN) return false;
    if (c->page_size != kPage || c->max_batch < 1 || c->max_batch > 64 || c->max_pages_per_seq < 1) return false;
    if (!(c->rms_eps > 0.f) || !(c->rope_theta > 1.f)) return false;
    if (c->head_layers < 0 || c->head_layers > GLANCE_MAX_HEAD_LAYERS) return false;
    for (int i = 0; i < c->head_layers && c->head_layers > 1; ++i) {
        if (c->head_taps[i] < 0 || c->head_taps[i] >= c->n_layers) return false;
        for (int j = 0; j < i; ++j)
            if (c->head_taps[j] == c->head_taps[i]) return false;
    }
    return true;
}

// head depth and the target layer each head layer taps
int head_depth(const glance_config &c) { return c.head_layers > 1 ? c.head_layers : 1; }
int head_tap(const glance_config &c, int i) { return c.head_layers > 1 ? c.head_taps[i] : c.n_layers - 1; }

}  // namespace

struct glance_ctx {
    float *ent_out = nullptr;               // device [max_batch]: root entropy written by every verify pass, or off
    bool ent_on = false;                    // the pass in flight is a verify pass (roots are rows s * N)
    bool sample_on = false;                 // the LM head of the pass in flight draws instead of taking the arg-max
    unsigned long long sample_seed = 0;
    float sample_inv_t = 1.f;
    glance_config cfg;
    Dims dims;
    Workspace ws;
    cudaStream_t stream;
    const bf16 *embed, *lm_head, *final_norm;
    std::vector<const bf16 *> ln1, wqkv, wo, ln2, wgu, wd;
    glance_head_weights head;
    std::vector<glance_head_layer> head_layer;   // all head layers, layer 0 first
    int64_t launches;
    // optional per-launch timing (event pairs created when profiling is first enabled)
    bool profiling = false;
    std::vector<cudaEvent_t> ev;      // 2 per tallied launch
    std::vector<double> ev_bytes;
    std::vector<int> ev_kind;
    size_t ev_used = 0;
    // TMA descriptors, keyed by (base, inner extent, rows, box rows); built on first use by a host-only call
    std::map<std::tuple<const void *, int, int, int>, CUtensorMap> maps;
    bool map_error = false;
    std::vector<double> inv_freq_host;   // staged for the one-time upload at creation
    // test hook: phase timestamps of successive GEMM launches, 16 words each, ring of trace_slots launches
    unsigned long long *trace = nullptr;
    int trace_slots = 0, trace_next = 0;
    // attention: which second bf16 terms the pure-context key tiles drop, and from which context length on
    int attn_lo_skip = 0, attn_lo_min_keys = 0;
    // test hook, one shot: the next glance_debug_gemm launch withholds one ring slot and waits at most this long
    int stall_kstep1 = 0;
    unsigned long long stall_limit_ns = 0;
};

namespace {

enum { KIND_GEMM = 0, KIND_ATTN = 1, KIND_SETUP = 2, KIND_CONTROL = 3, KIND_OTHER = 4, KIND_COUNT = 5 };

constexpr size_t kMaxProfiled = 32768;

inline bool prof_begin(glance_ctx *ctx) {
    const bool prof = ctx->profiling && ctx->ev_used < kMaxProfiled;
    if (prof) cudaEventRecord(ctx->ev[2 * ctx->ev_used], ctx->stream);
    return prof;
}
inline void prof_end(glance_ctx *ctx, bool prof, int kind, double bytes) {
    ctx->launches++;
    if (!prof) return;
    cudaEventRecord(ctx->ev[2 * ctx->ev_used + 1], ctx->stream);
    ctx->ev_bytes[ctx->ev_used] = bytes;
    ctx->ev_kind[ctx->ev_used] = kind;
    ctx->ev_used++;
}

#define LAUNCH(ctx, kind, call)                  \
    do {                                         \
        const bool prof_ = prof_begin(ctx);      \
        call;                                    \
        prof_end(ctx, prof_, kind, 0.0);         \
    } while (0)

const CUtensorMap *get_map(glance_ctx *ctx, const void *base, int inner, int rows, int box_rows) {
    auto key = std::make_tuple(base, inner, rows, box_rows);
    auto it = ctx->maps.find(key);
    if (it != ctx->maps.end()) return &it->second;
    CUtensorMap m;
    if (!tc_make_map(&m, base, (uint64_t)inner, (uint64_t)rows, (uint32_t)box_rows)) {
        ctx->map_error = true;
        return nullptr;
    }
    return &ctx->maps.emplace(key, m).first->second;
}

// Launches the weight-streaming GEMM described by `a` (mode: see gemm_tc.cuh) on X [R][K] (x_rows rows are
// allocated behind X) and W [Nout][K], and tallies its algorithmic bytes.
void gemm(glance_ctx *ctx, int mode, const bf16 *W, const bf16 *X, int x_rows, TcGemmArgs a) {
    const CUtensorMap *mw = get_map(ctx, W, a.K, a.Nout, mode == 1 ? 64 : 128);
    const CUtensorMap *mx = get_map(ctx, X, a.K, a.x_lo_row > 0 ? 2 * x_rows : x_rows, tc_row_pad(a.R));
    if (!mw || !mx) return;
    a.keys = ctx->ws.am_keys; a.counter = ctx->ws.am_counter; a.status = ctx->ws.status;
    if (ctx->trace && ctx->trace_slots > 0) {
        a.trace = ctx->trace + (size_t)(ctx->trace_next % ctx->trace_slots) * 16;
        ctx->trace_next++;
    }
    const bool prof = prof_begin(ctx);
    if (launch_gemm_tc(mode, a, *mw, *mx, ctx->stream) != cudaSuccess) ctx->map_error = true;
    // weights once, activations in (both planes when two-term), results out
    double bytes = 2.0 * a.Nout * a.K + (a.x_lo_row > 0 ? 4.0 : 2.0) * a.R * a.K;
    if (mode == 0) bytes += 4.0 * a.S * a.R * a.Nout;
    else if (mode == 1) bytes += (a.act_lo ? 4.0 : 2.0) * a.R * a.F;
    else if (mode == 2) bytes += 4.0 * a.R + (a.Y ? 4.0 * a.R * a.Nout : 0.0);
    else if (mode == 5) bytes += (a.Y ? 4.0 * a.R * a.Nout : 0.0) + 12.0 * a.R * ((a.Nout + 127) / 128);
    else if (mode == 3) bytes += (4.0 + 4.0 + (a.xb_lo ? 4.0 : 2.0)) * a.R * a.Nout;   // residual in/out + bf16 copy
    else bytes += 2.0 * a.R * a.Nout;
    prof_end(ctx, prof, KIND_GEMM, bytes);
}

// tree / block attention on one pool layer (K/V pages are fetched by TMA through a per-layer descriptor)
void attention(glance_ctx *ctx, AttnParams ap) {
    ap.trace = nullptr;
    if (ctx->trace && ctx->trace_slots > 0) {
        ap.trace = ctx->trace + (size_t)(ctx->trace_next % ctx->trace_slots) * 16;
        ctx->trace_next++;
    }
    const CUtensorMap *m = get_map(ctx, ap.pool_layer, ap.d, ap.geom.n_pages * 2 * ap.geom.n_kv_heads * kPage, kPage);
    if (!m) return;
    const bool prof = prof_begin(ctx);
    if (launch_attention_tc(ap, *m, ctx->stream) != cudaSuccess) ctx->map_error = true;
    prof_end(ctx, prof, KIND_ATTN, 0.0);
}

// row scales 1/rms from the per-tile sums of squares the producer left in ws.ssq
void with_row_scales(const glance_ctx *ctx, TcGemmArgs &a) {
    a.ssq = ctx->ws.ssq; a.n_ssq = ctx->dims.n_ssq; a.ssq_stride = ctx->dims.Rmax; a.eps = ctx->cfg.rms_eps;
}

struct LayerW {
    const bf16 *ln2, *wqkv, *wo, *wgu, *wd;
};

struct PassInfo {
    int R;                 // rows entering the layer
    int Rq;                // rows that continue after the K/V write (queries)
    int batch, T;          // attention: T query rows / extra keys per sequence
    const uint64_t *anc;   // or nullptr
    const glance_seqs *seqs;
    int seq_off;           // first sequence (prefill of one sequence of a batch)
};

KvGeom geom_of(const glance_ctx *ctx, const glance_seqs *s) {
    KvGeom g;
    g.n_pages = s->n_pages;
    g.n_kv_heads = ctx->cfg.n_kv_heads;
    g.head_dim = ctx->cfg.head_dim;
    g.max_pages_per_seq = ctx->cfg.max_pages_per_seq;
    return g;
}

RowMeta meta_of(const glance_ctx *ctx) {
    RowMeta m;
    m.seq = ctx->ws.row_seq;
    m.pos = ctx->ws.row_pos;
    m.kvrow = ctx->ws.row_kvrow;
    m.inv_freq = ctx->ws.inv_freq;
    m.rope_cos = ctx->ws.rope_cos;
    m.rope_sin = ctx->ws.rope_sin;
    return m;
}

RowOut rowout_of(const glance_ctx *ctx) {
    RowOut o;
    o.H = ctx->cfg.hidden;
    o.x = ctx->ws.x;
    o.xb = ctx->ws.xn;
    o.xb_lo = ctx->ws.xn + (size_t)ctx->dims.Rmax * ctx->cfg.hidden;
    o.ssq = ctx->ws.ssq;
    o.n_ssq = ctx->dims.n_ssq;
    o.ssq_stride = ctx->dims.Rmax;
    return o;
}

// One decoder layer over the rows of a pass: five launches.
//   QKV GEMM (+ 1/rms row scale, rotary, q / paged K,V write)  ->  attention  ->
//   O GEMM (+ residual, bf16 copy scaled by ln2, sums of squares)  ->
//   gate/up GEMM (+ 1/rms row scale, SwiGLU)  ->  down GEMM (+ residual, bf16 copy scaled by next_gain, sums of squares)
// On entry ws.x is the residual stream, ws.xn = bf16(x * gain) and ws.ssq its sums of squares; same on exit.
void run_layer(glance_ctx *ctx, const LayerW &w, bf16 *pool_layer, const PassInfo &ps, const bf16 *next_gain,
               bf16 *hidden_out) {
    const glance_config &c = ctx->cfg;
    const Dims &d = ctx->dims;
    Workspace &ws = ctx->ws;
    cudaStream_t st = ctx->stream;
    const KvGeom geom = geom_of(ctx, ps.seqs);
    const int32_t *page_table = ps.seqs->page_table + (size_t)ps.seq_off * c.max_pages_per_seq;
    const int32_t *seq_len = ps.seqs->seq_len + ps.seq_off;
    const int xr = d.Rmax;                             // rows allocated behind every activation buffer
    {
        TcGemmArgs g{};
        g.Nout = d.qkv_out; g.K = c.hidden; g.R = ps.R; g.S = choose_split(d.qkv_out, c.hidden, ps.R, false);
        with_row_scales(ctx, g);
        g.x_lo_row = 0;      // q, K, V are rounded to bf16 right after: the second term of x would buy nothing
        g.q = ws.q; g.q_lo = ws.q + (size_t)xr * d.qd; g.pool_layer = pool_layer; g.kvrow = ws.row_kvrow;
        g.v_off = (size_t)c.n_kv_heads * kPage * c.head_dim; g.head_stride = (size_t)kPage * c.head_dim;
        g.rope_cos = ws.rope_cos; g.rope_sin = ws.rope_sin;
        g.Hq = c.n_q_heads; g.Hkv = c.n_kv_heads; g.head_dim = c.head_dim; g.Rq = ps.Rq;
        gemm(ctx, 4, w.wqkv, ws.xn, xr, g);
    }
    if (ps.Rq == 0) return;
    AttnParams ap;
    ap.batch = ps.batch; ap.T = ps.T; ap.Hq = c.n_q_heads; ap.Hkv = c.n_kv_heads; ap.d = c.head_dim;
    ap.q = ws.q; ap.q_lo = ws.q + (size_t)xr * d.qd; ap.pool_layer = pool_layer; ap.geom = geom; ap.page_table = page_table; ap.seq_len = seq_len;
    ap.anc = ps.anc; ap.W = (ps.T + 63) / 64; ap.out = ws.attn; ap.out_lo = ws.attn + (size_t)xr * d.qd;
    ap.S = attention_tc_splits(ps.T, c.n_q_heads / c.n_kv_heads, c.n_kv_heads, ps.batch, c.head_dim);
    ap.status = ws.status;
    ap.lo_skip = ctx->attn_lo_skip; ap.lo_skip_min_keys = ctx->attn_lo_min_keys;
    attention(ctx, ap);
    const int R = ps.Rq;
    {
        TcGemmArgs g{};
        g.Nout = c.hidden; g.K = d.qd; g.R = R; g.S = choose_split(c.hidden, d.qd, R, true);
        g.x = ws.x; g.gain = w.ln2; g.xb = ws.xn; g.xb_lo = ws.xn + (size_t)xr * c.hidden; g.ssq_out = ws.ssq;
        g.ssq_stride = d.Rmax; g.x_lo_row = xr;
        gemm(ctx, 3, w.wo, ws.attn, xr, g);
    }
    {
        TcGemmArgs g{};
        g.Nout = 2 * c.ffn; g.K = c.hidden; g.R = R; g.S = 1; g.act = ws.act; g.act_lo = ws.act + (size_t)xr * c.ffn;
        g.F = c.ffn; g.x_lo_row = xr;
        with_row_scales(ctx, g);
        gemm(ctx, 1, w.wgu, ws.xn, xr, g);
    }
    {
        TcGemmArgs g{};
        g.Nout = c.hidden; g.K = c.ffn; g.R = R; g.S = choose_split(c.hidden, c.ffn, R, true);
        g.x = ws.x; g.gain = next_gain; g.xb = ws.xn; g.xb_lo = ws.xn + (size_t)xr * c.hidden; g.hidden_out = hidden_out;
        g.ssq_out = ws.ssq; g.ssq_stride = d.Rmax; g.x_lo_row = xr;
        gemm(ctx, 3, w.wd, ws.act, xr, g);
    }
}

// all target layers (+ LM head with fused arg-max) over rows prepared by a setup kernel
// `hidden_out` [head layers][ps.R][H]: slice i receives the residual stream after the target layer head layer i taps
void run_target(glance_ctx *ctx, const PassInfo &ps, bf16 *hidden_out, float *logits, int32_t *argmax) {
    const glance_config &c = ctx->cfg;
    const KvGeom geom = geom_of(ctx, ps.seqs);
    for (int l = 0; l < c.n_layers; ++l) {
        LayerW w{ctx->ln2[l], ctx->wqkv[l], ctx->wo[l], ctx->wgu[l], ctx->wd[l]};
        const bool last = (l + 1 == c.n_layers);
        bf16 *pool_layer = (bf16 *)ps.seqs->kv_pool + (size_t)l * geom.layer_stride();
        bf16 *tap_out = nullptr;
        for (int i = 0; i < head_depth(c) && hidden_out; ++i)
            if (head_tap(c, i) == l) tap_out = hidden_out + (size_t)i * ps.R * c.hidden;
        run_layer(ctx, w, pool_layer, ps, last ? ctx->final_norm : ctx->ln1[l + 1], tap_out);
    }
    if (argmax) {   // logits are stored only on request
        TcGemmArgs g{};
        g.Nout = c.vocab; g.K = c.hidden; g.R = ps.R; g.S = 1; g.Y = logits; g.ldy = c.vocab; g.argmax = argmax;
        g.x_lo_row = 0;      // logits only decide an arg-max / top-k: one term is enough
        if (ctx->sample_on) {
            g.sample_pos = ctx->ws.row_pos; g.sample_seed = ctx->sample_seed; g.sample_inv_t = ctx->sample_inv_t;
        }
        if (ctx->ent_on && ctx->ent_out) {
            g.ent_out = ctx->ent_out; g.ent_part = ctx->ws.ent_part; g.ent_N = ps.T; g.ent_batch = ps.batch;
        }
        with_row_scales(ctx, g);
        gemm(ctx, 2, ctx->lm_head, ctx->ws.xn, ctx->dims.Rmax, g);
    }
}

int32_t check_seqs(const glance_ctx *ctx, const glance_seqs *s) {
    if (!ctx || !s) return GLANCE_E_INVALID_ARG;
    if (s->batch < 1 || s->batch > ctx->cfg.max_batch || s->n_pages < 1) return GLANCE_E_INVALID_ARG;
    if (!s->seq_len || !s->root || !s->page_table || !s->kv_pool || !s->head_kv_pool || !s->feat || !s->feat_count)
        return GLANCE_E_INVALID_ARG;
    return GLANCE_OK;
}

int32_t finish(glance_ctx *ctx) {
    if (ctx->map_error) {
        ctx->map_error = false;
        return GLANCE_E_CUDA;
    }
    return cudaPeekAtLastError() == cudaSuccess ? GLANCE_OK : GLANCE_E_CUDA;
}

__global__ void set_seq_kernel(int32_t *seq_len, int32_t *root, int32_t len, int32_t r) {
    *seq_len = len;
    *root = r;
}

}  // namespace

extern "C" {

const char *glance_status_string(int32_t status) {
    switch (status) {
        case GLANCE_OK: return "ok";
        case GLANCE_E_INVALID_ARG: return "invalid argument";
        case GLANCE_E_SHAPE: return "unsupported shape";
        case GLANCE_E_CAPACITY: return "capacity exceeded";
        case GLANCE_E_CUDA: return "CUDA error";
        case GLANCE_E_TIMEOUT: return "device wait timed out";
        case GLANCE_E_BOUNDS: return "device index out of bounds";
        case GLANCE_E_STATE: return "invalid call order";
        default: return "unknown status";
    }
}

size_t glance_workspace_bytes(const glance_config *cfg) {
    if (!config_ok(cfg)) return 0;
    return carve(*cfg, make_dims(*cfg), nullptr).total;
}

int32_t glance_create(const glance_config *cfg, const glance_target_weights *t, const glance_head_weights *h,
                      void *workspace, size_t workspace_bytes, void *cuda_stream, glance_ctx **out) {
    if (!cfg || !t || !h || !workspace || !out) return GLANCE_E_INVALID_ARG;
    if (!config_ok(cfg)) return GLANCE_E_SHAPE;
    if (((uintptr_t)workspace & 255) != 0) return GLANCE_E_INVALID_ARG;
    if (!t->embed || !t->lm_head || !t->final_norm || !t->ln1 || !t->wqkv || !t->wo || !t->ln2 || !t->wgu || !t->wd)
        return GLANCE_E_INVALID_ARG;
    if (!h->mask_embed || !h->ctx_norm || !h->ln1 || !h->wqkv || !h->wo || !h->ln2 || !h->wgu || !h->wd ||
        !h->final_norm)
        return GLANCE_E_INVALID_ARG;
    const Dims d = make_dims(*cfg);
    Workspace ws = carve(*cfg, d, (unsigned char *)workspace);
    if (ws.total > workspace_bytes) return GLANCE_E_CAPACITY;
    glance_ctx *ctx = new (std::nothrow) glance_ctx();
    if (!ctx) return GLANCE_E_INVALID_ARG;
    ctx->cfg = *cfg;
    ctx->dims = d;
    ctx->ws = ws;
    ctx->stream = (cudaStream_t)cuda_stream;
    ctx->embed = (const bf16 *)t->embed;
    ctx->lm_head = (const bf16 *)t->lm_head;
    ctx->final_norm = (const bf16 *)t->final_norm;
    for (int l = 0; l < cfg->n_layers; ++l) {
        if (!t->ln1[l] || !t->wqkv[l] || !t->wo[l] || !t->ln2[l] || !t->wgu[l] || !t->wd[l]) {
            delete ctx;
            return GLANCE_E_INVALID_ARG;
        }
        ctx->ln1.push_back((const bf16 *)t->ln1[l]);
        ctx->wqkv.push_back((const bf16 *)t->wqkv[l]);
        ctx->wo.push_back((const bf16 *)t->wo[l]);
        ctx->ln2.push_back((const bf16 *)t->ln2[l]);
        ctx->wgu.push_back((const bf16 *)t->wgu[l]);
        ctx->wd.push_back((const bf16 *)t->wd[l]);
    }
    ctx->head = *h;
    ctx->head_layer.push_back(glance_head_layer{h->ctx_norm, h->ln1, h->wqkv, h->wo, h->ln2, h->wgu, h->wd});
    for (int i = 1; i < head_depth(*cfg); ++i) {
        const glance_head_layer *m = h->more ? &h->more[i - 1] : nullptr;
        if (!m || !m->ctx_norm || !m->ln1 || !m->wqkv || !m->wo || !m->ln2 || !m->wgu || !m->wd) {
            delete ctx;
            return GLANCE_E_INVALID_ARG;
        }
        ctx->head_layer.push_back(*m);
    }
    ctx->launches = 0;
    // rotary frequencies theta^(-2i/d) in double, uploaded once
    ctx->inv_freq_host.resize(cfg->head_dim / 2);
    for (int i = 0; i < cfg->head_dim / 2; ++i)
        ctx->inv_freq_host[i] = std::pow((double)cfg->rope_theta, -(2.0 * i) / (double)cfg->head_dim);
    if (cudaMemcpyAsync(ws.inv_freq, ctx->inv_freq_host.data(), ctx->inv_freq_host.size() * 8, cudaMemcpyHostToDevice,
                        ctx->stream) != cudaSuccess) {
        delete ctx;
        return GLANCE_E_CUDA;
    }
    // counters and the status word start at zero
    if (cudaMemsetAsync(ws.walk_ctr, 0, (size_t)cfg->max_batch * 4, ctx->stream) != cudaSuccess ||
        cudaMemsetAsync(ws.status, 0, 256, ctx->stream) != cudaSuccess ||
        cudaMemsetAsync(ws.am_keys, 0, (size_t)d.Rlog * 8, ctx->stream) != cudaSuccess ||
        cudaMemsetAsync(ws.am_counter, 0, 256, ctx->stream) != cudaSuccess ||
        cudaMemsetAsync(ws.tk_thr, 0, (size_t)cfg->max_batch * cfg->block_B * kTopkTileCap * 4, ctx->stream) != cudaSuccess) {
        delete ctx;
        return GLANCE_E_CUDA;
    }
    *out = ctx;
    return GLANCE_OK;
}

int32_t glance_destroy(glance_ctx *ctx) {
    if (!ctx) return GLANCE_E_INVALID_ARG;
    for (auto &e : ctx->ev) cudaEventDestroy(e);
    delete ctx;
    return GLANCE_OK;
}

int32_t glance_prefill(glance_ctx *ctx, const glance_seqs *seqs, int32_t seq, const void *embeds, const int32_t *ids,
                       int32_t count) {
    int32_t rc = check_seqs(ctx, seqs);
    if (rc) return rc;
    if (seq < 0 || seq >= seqs->batch || count < 1) return GLANCE_E_INVALID_ARG;
    if ((embeds == nullptr) == (ids == nullptr)) return GLANCE_E_INVALID_ARG;
    const glance_config &c = ctx->cfg;
    Workspace &ws = ctx->ws;
    cudaStream_t st = ctx->stream;
    const int N = c.tree_N;
    for (int done = 0; done < count; done += N) {
        const int n = std::min(N, count - done);
        const bool last = (done + n == count);
        const KvGeom tg = geom_of(ctx, seqs);
        const int32_t *pt = seqs->page_table + (size_t)seq * c.max_pages_per_seq;
        VerifySetup vs{};
        vs.batch = 1; vs.N = N; vs.d = c.head_dim; vs.theta = c.rope_theta;
        vs.seq_len = seqs->seq_len + seq; vs.token = nullptr; vs.depth = nullptr;
        vs.row_embeds = embeds ? (const bf16 *)embeds + (size_t)done * c.hidden : nullptr;
        vs.row_ids = ids ? ids + done : nullptr;
        vs.count = n; vs.chain_anc = ws.chain_anc; vs.embed = ctx->embed; vs.gain = ctx->ln1[0]; vs.vocab = c.vocab;
        vs.capacity = c.max_pages_per_seq * kPage; vs.geom = tg; vs.page_table = pt; vs.out = rowout_of(ctx);
        vs.meta = meta_of(ctx); vs.status = ws.status;
        LAUNCH(ctx, KIND_SETUP, launch_setup_verify(vs, st));
        PassInfo ps{N, N, 1, N, ws.chain_anc, seqs, seq};
        run_target(ctx, ps, ws.hidden_tmp, nullptr, last ? ws.argmax_tmp : nullptr);
        // head context K/V of the new positions (Section 3.2: keys and values are the target's hidden states): every
        // head layer projects the hidden states of the target layer it taps with its own weights into its own pool
        for (int i = 0; i < head_depth(c); ++i) {
            const glance_head_layer &hl = ctx->head_layer[i];
            DraftSetup ds{};
            ds.batch = 1; ds.B = c.block_B; ds.FR = N; ds.d = c.head_dim; ds.theta = c.rope_theta;
            ds.seq_len = seqs->seq_len + seq; ds.root = seqs->root + seq;
            ds.feat = ws.hidden_tmp + (size_t)i * N * c.hidden; ds.feat_count = nullptr;
            ds.count_const = n; ds.n_block = 0; ds.embed = ctx->embed; ds.mask_embed = (const bf16 *)ctx->head.mask_embed;
            ds.gain_block = (const bf16 *)hl.ln1; ds.gain_feat = (const bf16 *)hl.ctx_norm;
            ds.vocab = c.vocab; ds.capacity = c.max_pages_per_seq * kPage; ds.geom = tg; ds.page_table = pt;
            ds.out = rowout_of(ctx); ds.meta = meta_of(ctx); ds.status = ws.status;
            LAUNCH(ctx, KIND_SETUP, launch_setup_draft(ds, st));
            LayerW hw{(const bf16 *)hl.ln2, (const bf16 *)hl.wqkv, (const bf16 *)hl.wo, (const bf16 *)hl.wgu,
                      (const bf16 *)hl.wd};
            PassInfo hp{N, 0, 1, N, nullptr, seqs, seq};
            run_layer(ctx, hw, (bf16 *)seqs->head_kv_pool + (size_t)i * tg.layer_stride(), hp, nullptr, nullptr);
        }
        LAUNCH(ctx, KIND_CONTROL, launch_prefill_advance(seqs->seq_len + seq, seqs->root + seq, seqs->feat_count + seq,
                                                         last ? ws.argmax_tmp : nullptr, n, st));
    }
    return finish(ctx);
}

int32_t glance_seq_truncate(glance_ctx *ctx, const glance_seqs *seqs, int32_t seq, int32_t new_len, int32_t new_root) {
    int32_t rc = check_seqs(ctx, seqs);
    if (rc) return rc;
    if (seq < 0 || seq >= seqs->batch || new_len < 0 || new_root < 0 || new_root >= ctx->cfg.vocab)
        return GLANCE_E_INVALID_ARG;
    LAUNCH(ctx, KIND_CONTROL, (set_seq_kernel<<<1, 1, 0, ctx->stream>>>(seqs->seq_len + seq, seqs->root + seq, new_len, new_root)));
    return finish(ctx);
}

int32_t glance_draft_block(glance_ctx *ctx, const glance_seqs *seqs, int32_t *topk_ids, float *topk_lp,
                           float *logits_dbg) {
    int32_t rc = check_seqs(ctx, seqs);
    if (rc) return rc;
    if (!topk_ids || !topk_lp) return GLANCE_E_INVALID_ARG;
    const glance_config &c = ctx->cfg;
    Workspace &ws = ctx->ws;
    cudaStream_t st = ctx->stream;
    const int batch = seqs->batch, B = c.block_B;
    const int R1 = batch * B, R = 2 * R1;
    const KvGeom hgeom = geom_of(ctx, seqs);
    const int HL = head_depth(c);
    for (int i = 0; i < HL; ++i) {
        // head layer i: block rows (from the embeddings, or from the layer below) and the feature rows of the
        // positions committed last, taken from the target layer this head layer taps
        const glance_head_layer &hl = ctx->head_layer[i];
        DraftSetup ds{};
        ds.batch = batch; ds.B = B; ds.FR = B; ds.d = c.head_dim; ds.theta = c.rope_theta;
        ds.seq_len = seqs->seq_len; ds.root = seqs->root;
        ds.feat = (const bf16 *)seqs->feat + (size_t)i * batch * B * c.hidden;
        ds.feat_count = seqs->feat_count; ds.count_const = 0; ds.n_block = B; ds.features_only = i > 0 ? 1 : 0;
        ds.embed = ctx->embed; ds.mask_embed = (const bf16 *)ctx->head.mask_embed;
        // block rows use the head layer's input norm, feature rows its context norm
        ds.gain_block = (const bf16 *)hl.ln1; ds.gain_feat = (const bf16 *)hl.ctx_norm; ds.vocab = c.vocab;
        ds.capacity = c.max_pages_per_seq * kPage; ds.geom = hgeom; ds.page_table = seqs->page_table;
        ds.out = rowout_of(ctx); ds.meta = meta_of(ctx); ds.status = ws.status;
        LAUNCH(ctx, KIND_SETUP, launch_setup_draft(ds, st));
        LayerW hw{(const bf16 *)hl.ln2, (const bf16 *)hl.wqkv, (const bf16 *)hl.wo, (const bf16 *)hl.wgu, (const bf16 *)hl.wd};
        PassInfo ps{R, R1, batch, B, nullptr, seqs, 0};
        const bf16 *next_gain = i + 1 < HL ? (const bf16 *)ctx->head_layer[i + 1].ln1 : (const bf16 *)ctx->head.final_norm;
        run_layer(ctx, hw, (bf16 *)seqs->head_kv_pool + (size_t)i * hgeom.layer_stride(), ps, next_gain, nullptr);
    }
    // LM head over the block rows with the per-offset top-k fused into its epilogue: every 128-feature tile leaves
    // its log-sum-exp share and the keys that can still be among a row's k largest; one small launch merges them.
    // The logits themselves are written only on request.
    {
        TcGemmArgs g{};
        g.Nout = c.vocab; g.K = c.hidden; g.R = R1; g.S = 1; g.Y = logits_dbg; g.ldy = c.vocab; g.split_stride = 0;
        g.x_lo_row = 0;
        g.tk_k = c.topk; g.tk_B = B; g.tk_thr = ws.tk_thr; g.tk_ml = ws.tk_ml; g.tk_cnt = ws.tk_cnt; g.tk_cand = ws.tk_cand;
        with_row_scales(ctx, g);
        gemm(ctx, 5, ctx->lm_head, ws.xn, ctx->dims.Rmax, g);
    }
    LAUNCH(ctx, KIND_CONTROL, launch_topk_merge(batch, B, (c.vocab + 127) / 128, c.topk, ws.tk_thr, ws.tk_ml, ws.tk_cnt,
                                                ws.tk_cand, topk_ids, topk_lp, st));
    return finish(ctx);
}

int32_t glance_build_tree(glance_ctx *ctx, int32_t batch, const int32_t *root, const int32_t *topk_ids,
                          const float *topk_lp, const glance_tree *out) {
    if (!ctx || !root || !topk_ids || !topk_lp || !out) return GLANCE_E_INVALID_ARG;
    if (batch < 1 || batch > ctx->cfg.max_batch) return GLANCE_E_INVALID_ARG;
    if (!out->token || !out->parent || !out->depth || !out->rank || !out->score || !out->anc || !out->n_nodes)
        return GLANCE_E_INVALID_ARG;
    const glance_config &c = ctx->cfg;
    LAUNCH(ctx, KIND_CONTROL, launch_build_tree(batch, c.tree_N, c.block_B - 1, c.topk, root, topk_ids, topk_lp, *out, ctx->stream));
    return finish(ctx);
}

static int32_t verify_common(glance_ctx *ctx, const glance_seqs *seqs, const glance_tree *tree, int32_t *decisions,
                             void *hidden, float *logits_dbg) {
    int32_t rc = check_seqs(ctx, seqs);
    if (rc) return rc;
    if (!tree || !tree->token || !tree->depth || !tree->anc || !decisions || !hidden) return GLANCE_E_INVALID_ARG;
    const glance_config &c = ctx->cfg;
    Workspace &ws = ctx->ws;
    const int batch = seqs->batch, N = c.tree_N;
    VerifySetup vs{};
    vs.batch = batch; vs.N = N; vs.d = c.head_dim; vs.theta = c.rope_theta;
    vs.seq_len = seqs->seq_len; vs.token = tree->token; vs.depth = tree->depth; vs.row_embeds = nullptr;
    vs.row_ids = nullptr; vs.count = 0; vs.chain_anc = nullptr; vs.embed = ctx->embed; vs.gain = ctx->ln1[0];
    vs.vocab = c.vocab; vs.capacity = c.max_pages_per_seq * kPage; vs.geom = geom_of(ctx, seqs);
    vs.page_table = seqs->page_table; vs.out = rowout_of(ctx); vs.meta = meta_of(ctx); vs.status = ws.status;
    LAUNCH(ctx, KIND_SETUP, launch_setup_verify(vs, ctx->stream));
    PassInfo ps{batch * N, batch * N, batch, N, tree->anc, seqs, 0};
    ctx->ent_on = true;
    run_target(ctx, ps, (bf16 *)hidden, logits_dbg, decisions);
    ctx->ent_on = false;
    return finish(ctx);
}

int32_t glance_verify_tree(glance_ctx *ctx, const glance_seqs *seqs, const glance_tree *tree, int32_t *argmax,
                           void *hidden, float *logits_dbg) {
    if (!ctx) return GLANCE_E_INVALID_ARG;
    ctx->sample_on = false;
    return verify_common(ctx, seqs, tree, argmax, hidden, logits_dbg);
}

int32_t glance_verify_tree_sample(glance_ctx *ctx, const glance_seqs *seqs, const glance_tree *tree, uint64_t seed,
                                  float temperature, int32_t *draws, void *hidden, float *logits_dbg) {
    if (!ctx || !(temperature > 0.f)) return GLANCE_E_INVALID_ARG;
    ctx->sample_on = true;
    ctx->sample_seed = seed;
    ctx->sample_inv_t = 1.f / temperature;
    const int32_t rc = verify_common(ctx, seqs, tree, draws, hidden, logits_dbg);
    ctx->sample_on = false;
    return rc;
}

static int32_t commit_common(glance_ctx *ctx, const glance_seqs *seqs, WalkCommit &wc, const void *hidden) {
    const glance_config &c = ctx->cfg;
    wc.batch = seqs->batch; wc.N = c.tree_N; wc.B = c.block_B; wc.H = c.hidden; wc.n_layers = c.n_layers;
    wc.hidden = (const bf16 *)hidden; wc.kv_pool = (bf16 *)seqs->kv_pool; wc.geom = geom_of(ctx, seqs);
    wc.page_table = seqs->page_table; wc.seq_len = seqs->seq_len; wc.root = seqs->root;
    wc.feat_count = seqs->feat_count; wc.feat = (bf16 *)seqs->feat; wc.counters = ctx->ws.walk_ctr;
    wc.n_taps = head_depth(c);
    wc.status = ctx->ws.status;
    LAUNCH(ctx, KIND_CONTROL, launch_walk_commit(wc, ctx->stream));
    return finish(ctx);
}

int32_t glance_accept_commit(glance_ctx *ctx, const glance_seqs *seqs, const glance_tree *tree, const int32_t *argmax,
                             const void *hidden, int32_t *accept_len, int32_t *path, int32_t *out_tokens) {
    int32_t rc = check_seqs(ctx, seqs);
    if (rc) return rc;
    if (!tree || !tree->token || !tree->parent || !tree->n_nodes || !argmax || !hidden || !accept_len || !path ||
        !out_tokens)
        return GLANCE_E_INVALID_ARG;
    WalkCommit wc{};
    wc.token = tree->token; wc.parent = tree->parent; wc.n_nodes = tree->n_nodes; wc.argmax = argmax;
    wc.accept_len = accept_len; wc.path = path; wc.out_tokens = out_tokens;
    return commit_common(ctx, seqs, wc, hidden);
}

int32_t glance_commit_forced(glance_ctx *ctx, const glance_seqs *seqs, const void *hidden, const int32_t *path,
                             const int32_t *path_len, const int32_t *new_root) {
    int32_t rc = check_seqs(ctx, seqs);
    if (rc) return rc;
    if (!hidden || !path || !path_len || !new_root) return GLANCE_E_INVALID_ARG;
    WalkCommit wc{};
    wc.forced_path = path; wc.forced_len = path_len; wc.forced_root = new_root;
    return commit_common(ctx, seqs, wc, hidden);
}

int32_t glance_log_root_entropy(glance_ctx *ctx, float *entropy) {
    if (!ctx) return GLANCE_E_INVALID_ARG;
    ctx->ent_out = entropy;
    return GLANCE_OK;
}

int32_t glance_poll_status(glance_ctx *ctx, int32_t *device_status) {
    if (!ctx || !device_status) return GLANCE_E_INVALID_ARG;
    int32_t v = 0;
    if (cudaMemcpyAsync(&v, ctx->ws.status, 4, cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess) return GLANCE_E_CUDA;
    if (cudaMemsetAsync(ctx->ws.status, 0, 4, ctx->stream) != cudaSuccess) return GLANCE_E_CUDA;
    if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return GLANCE_E_CUDA;
    *device_status = v;
    return GLANCE_OK;
}

int32_t glance_debug_attention(glance_ctx *ctx, const glance_seqs *seqs, int32_t layer, const void *q,
                               const void *q_lo, const uint64_t *anc, int32_t T, void *out, void *out_lo) {
    int32_t rc = check_seqs(ctx, seqs);
    if (rc) return rc;
    const glance_config &c = ctx->cfg;
    if (!q || !out || layer < 0 || layer >= c.n_layers || T < 1 || T > std::max(c.tree_N, c.block_B))
        return GLANCE_E_INVALID_ARG;
    const KvGeom geom = geom_of(ctx, seqs);
    AttnParams ap;
    ap.batch = seqs->batch; ap.T = T; ap.Hq = c.n_q_heads; ap.Hkv = c.n_kv_heads; ap.d = c.head_dim;
    ap.q = (const bf16 *)q; ap.q_lo = (const bf16 *)q_lo; ap.pool_layer = (const bf16 *)seqs->kv_pool + (size_t)layer * geom.layer_stride();
    ap.geom = geom; ap.page_table = seqs->page_table; ap.seq_len = seqs->seq_len; ap.anc = anc; ap.W = (T + 63) / 64;
    ap.out = (bf16 *)out; ap.out_lo = (bf16 *)out_lo; ap.S = attention_tc_splits(T, c.n_q_heads / c.n_kv_heads, c.n_kv_heads, seqs->batch, c.head_dim);
    ap.status = ctx->ws.status;
    ap.lo_skip = ctx->attn_lo_skip; ap.lo_skip_min_keys = ctx->attn_lo_min_keys;
    attention(ctx, ap);
    return finish(ctx);
}

int32_t glance_debug_gemm(glance_ctx *ctx, int32_t mode, const void *W, const void *X, float *Y, void *act,
                             int32_t *argmax, int32_t Nout, int32_t K, int32_t R, int32_t S) {
    if (!ctx || !W || !X || mode < 0 || mode > 2) return GLANCE_E_INVALID_ARG;
    if (Nout < 1 || K < 64 || K % 64 || R < 1 || R > ctx->dims.Rlog || S < 1 || S > 16) return GLANCE_E_INVALID_ARG;
    if ((mode == 0 && !Y) || (mode == 1 && (!act || Nout % 2)) || (mode == 2 && !argmax)) return GLANCE_E_INVALID_ARG;
    TcGemmArgs g{};
    g.Nout = Nout; g.K = K; g.R = R; g.S = mode == 0 ? S : 1; g.Y = Y; g.ldy = Nout; g.split_stride = (size_t)R * Nout;
    g.act = (bf16 *)act; g.F = Nout / 2; g.argmax = argmax;
    g.stall_kstep1 = ctx->stall_kstep1; g.wait_limit_ns = ctx->stall_limit_ns;
    ctx->stall_kstep1 = 0; ctx->stall_limit_ns = 0;      // one shot
    gemm(ctx, mode, (const bf16 *)W, (const bf16 *)X, R, g);
    // the hook's operands are transient: their two descriptors are dropped again, everybody else's stay
    ctx->maps.erase(std::make_tuple((const void *)W, K, Nout, mode == 1 ? 64 : 128));
    ctx->maps.erase(std::make_tuple((const void *)X, K, R, tc_row_pad(R)));
    return finish(ctx);
}

int32_t glance_debug_stall_next_gemm(glance_ctx *ctx, int32_t kstep, uint64_t wait_limit_ns) {
    if (!ctx || kstep < 0 || wait_limit_ns < 1000 || wait_limit_ns > 1000ull * 1000ull * 1000ull) return GLANCE_E_INVALID_ARG;
    ctx->stall_kstep1 = kstep + 1;
    ctx->stall_limit_ns = wait_limit_ns;
    return GLANCE_OK;
}

int32_t glance_debug_attention_terms(glance_ctx *ctx, int32_t lo_skip, int32_t min_keys) {
    if (!ctx || lo_skip < 0 || lo_skip > 3 || min_keys < 0) return GLANCE_E_INVALID_ARG;
    ctx->attn_lo_skip = lo_skip;
    ctx->attn_lo_min_keys = min_keys;
    return GLANCE_OK;
}

int32_t glance_debug_trace(glance_ctx *ctx, uint64_t *buffer, int32_t slots) {
    if (!ctx || slots < 0 || (buffer == nullptr) != (slots == 0)) return GLANCE_E_INVALID_ARG;
    ctx->trace = (unsigned long long *)buffer;
    ctx->trace_slots = slots;
    ctx->trace_next = 0;
    return GLANCE_OK;
}

int32_t glance_profile_enable(glance_ctx *ctx, int32_t on) {
    if (!ctx) return GLANCE_E_INVALID_ARG;
    if (on && ctx->ev.empty()) {
        ctx->ev.resize(2 * kMaxProfiled);
        ctx->ev_bytes.resize(kMaxProfiled);
        ctx->ev_kind.resize(kMaxProfiled);
        for (auto &e : ctx->ev)
            if (cudaEventCreate(&e) != cudaSuccess) return GLANCE_E_CUDA;
    }
    ctx->profiling = on != 0;     // the tally survives pauses; glance_profile_read resets it
    return GLANCE_OK;
}

int32_t glance_profile_read(glance_ctx *ctx, double *ms, double *bytes, int64_t *launches) {
    if (!ctx || !ms || !bytes || !launches) return GLANCE_E_INVALID_ARG;
    if (ctx->ev.empty()) return GLANCE_E_STATE;       // nothing was ever tallied: glance_profile_enable comes first
    if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return GLANCE_E_CUDA;
    for (int k = 0; k < KIND_COUNT; ++k) { ms[k] = 0.0; bytes[k] = 0.0; launches[k] = 0; }
    for (size_t i = 0; i < ctx->ev_used; ++i) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, ctx->ev[2 * i], ctx->ev[2 * i + 1]) != cudaSuccess) return GLANCE_E_CUDA;
        const int k = ctx->ev_kind[i];
        ms[k] += t;
        bytes[k] += ctx->ev_bytes[i];
        launches[k]++;
    }
    ctx->ev_used = 0;
    return GLANCE_OK;
}

int64_t glance_launch_count(const glance_ctx *ctx) { return ctx ? ctx->launches : 0; }

}  // extern "C"
