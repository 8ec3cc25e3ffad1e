// Row setup kernels of the verify and draft passes (embedding gather, rotary table, paged row offsets, first
// norm statistics) and the two-stage per-offset top-k + log-softmax of the draft pass.
#include "gemm_tc.cuh"
#include "kernels.cuh"
#include "tc_ptx.cuh"

namespace glance {

// ------------------------------------------------------------------------------------------
// Row setup shared by the verify and draft passes.  One block per row:
//   * rotary table of the row: angle = pos * theta^(-2i/d), argument reduction in double
//   * element offset of the row's K slot (kv head 0) inside a layer of the paged pool
//   * fp32 residual row x, its bf16 copy scaled by the first norm's gain, and its sum of squares
//     (the consumer GEMM multiplies its results by 1/rms, so no separate normalisation pass exists)
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void fill_rope_row(const RowMeta &m, int r, int pos, int d, float theta) {
    // angle = pos * theta^(-2i/d): the product and its reduction modulo 2 pi are done in double (a handful of
    // FP64 instructions) with the per-dimension frequencies precomputed in double on the host; the reduced
    // angle lies in [-pi, pi], where single-precision sincos is accurate to ~1e-7.
    (void)theta;
    const int half = d >> 1;
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        const double x = (double)pos * m.inv_freq[i];
        const double k = rint(x * 0.15915494309189535);           // 1 / (2 pi)
        const double red = fma(-k, 1.2246467991473532e-16 * 2.0, fma(-k, 6.283185307179586, x));
        float s, c;
        sincosf((float)red, &s, &c);
        m.rope_cos[(size_t)r * half + i] = c;
        m.rope_sin[(size_t)r * half + i] = s;
    }
}

__device__ __forceinline__ long long kv_row_offset(const KvGeom &g, const int32_t *page_table, int s, int slot_pos,
                                                   int32_t *status) {
    if (slot_pos < 0) return -1;
    const int pg = slot_pos / kPage;
    if (pg >= g.max_pages_per_seq) { set_status(status, GLANCE_E_BOUNDS); return -1; }
    const int page = page_table[(size_t)s * g.max_pages_per_seq + pg];
    if (page < 0 || page >= g.n_pages) { set_status(status, GLANCE_E_BOUNDS); return -1; }
    return (long long)g.row(page, 0, 0, slot_pos % kPage);
}

// x[c] = src[c] (or 0), xb[c] = bf16(x[c] * gain[c]), ssq[0][r] = sum x^2, ssq[i>0][r] = 0
__device__ __forceinline__ void emit_row(const RowOut &o, int r, const bf16 *src, const bf16 *gain) {
    // H is a multiple of 64: the row is handled in 16-byte groups of eight bf16, up to four groups per thread
    // with all loads issued before the first use (the source row usually comes from HBM)
    __shared__ float red[4];
    float *x = o.x + (size_t)r * o.H;
    bf16 *xb = o.xb + (size_t)r * o.H;
    bf16 *xl = o.xb_lo ? o.xb_lo + (size_t)r * o.H : nullptr;
    const int groups = o.H >> 3;
    float ss = 0.f;
    for (int g0 = threadIdx.x; g0 < groups; g0 += 4 * blockDim.x) {
        uint4 raw[4], gn[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int g = g0 + u * blockDim.x;
            raw[u] = make_uint4(0, 0, 0, 0);
            gn[u] = make_uint4(0, 0, 0, 0);
            if (g < groups) {
                if (src) raw[u] = *reinterpret_cast<const uint4 *>(src + g * 8);
                gn[u] = *reinterpret_cast<const uint4 *>(gain + g * 8);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int g = g0 + u * blockDim.x;
            if (g >= groups) continue;
            const __nv_bfloat162 *v2 = reinterpret_cast<const __nv_bfloat162 *>(&raw[u]);
            const __nv_bfloat162 *g2 = reinterpret_cast<const __nv_bfloat162 *>(&gn[u]);
            float f[8], sg[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                f[2 * j] = __low2float(v2[j]);
                f[2 * j + 1] = __high2float(v2[j]);
                sg[2 * j] = f[2 * j] * __low2float(g2[j]);
                sg[2 * j + 1] = f[2 * j + 1] * __high2float(g2[j]);
                ss += f[2 * j] * f[2 * j] + f[2 * j + 1] * f[2 * j + 1];
            }
            *reinterpret_cast<float4 *>(x + g * 8) = make_float4(f[0], f[1], f[2], f[3]);
            *reinterpret_cast<float4 *>(x + g * 8 + 4) = make_float4(f[4], f[5], f[6], f[7]);
            tc::store_two_term(xb + g * 8, xl ? xl + g * 8 : nullptr, make_float4(sg[0], sg[1], sg[2], sg[3]));
            tc::store_two_term(xb + g * 8 + 4, xl ? xl + g * 8 + 4 : nullptr, make_float4(sg[4], sg[5], sg[6], sg[7]));
        }
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        o.ssq[r] = ((red[0] + red[1]) + red[2]) + red[3];
        for (int i = 1; i < o.n_ssq; ++i) o.ssq[(size_t)i * o.ssq_stride + r] = 0.f;
    }
}

// Verify-pass rows (Algorithm 1 line 3: pack the root and the tree).  Row r = s*N + i is node i of
// sequence s at rotary position P + depth[i]; its K/V go to cache row P + i.  In prefill mode the rows are
// a causal chain of `count` given embeddings / token ids and the chain's ancestor mask is emitted.
__global__ void __launch_bounds__(128) setup_verify_kernel(VerifySetup p) {
    const int r = blockIdx.x;
    const int s = r / p.N, i = r % p.N;
    const int P = p.seq_len[s];
    const bool prefill = (p.token == nullptr);
    int depth = prefill ? i : p.depth[r];
    if (!prefill && (depth < 0 || depth > kMaxBlock)) depth = 0;
    if (threadIdx.x == 0) {
        // a sequence without room for its N rows is reported once, as a capacity fault, and writes no K/V at all
        const bool fits = P >= 0 && P + p.N <= p.capacity;
        if (!fits) set_status(p.status, GLANCE_E_CAPACITY);
        p.meta.seq[r] = s;
        p.meta.pos[r] = P + depth;
        p.meta.kvrow[r] = fits ? kv_row_offset(p.geom, p.page_table, s, P + i, p.status) : -1;
    }
    fill_rope_row(p.meta, r, P + depth, p.d, p.theta);
    const bf16 *src = nullptr;
    if (prefill) {
        if (i < p.count) {
            if (p.row_embeds) src = p.row_embeds + (size_t)i * p.out.H;
            else {
                int t = p.row_ids[i];
                if (t < 0 || t >= p.vocab) { t = 0; if (threadIdx.x == 0) set_status(p.status, GLANCE_E_BOUNDS); }
                src = p.embed + (size_t)t * p.out.H;
            }
        }
        // causal chain mask: row i sees rows 0..i
        const int W = (p.N + 63) >> 6;
        if (threadIdx.x < W) {
            int w = threadIdx.x;
            uint64_t bits;
            if (i >= 64 * (w + 1) - 1) bits = ~0ull;
            else if (i < 64 * w) bits = 0ull;
            else bits = (~0ull) >> (63 - (i - 64 * w));
            p.chain_anc[(size_t)i * W + w] = bits;
        }
    } else {
        int t = p.token[r];
        if (t < 0 || t >= p.vocab) { t = 0; if (threadIdx.x == 0) set_status(p.status, GLANCE_E_BOUNDS); }
        src = p.embed + (size_t)t * p.out.H;
    }
    emit_row(p.out, r, src, p.gain);
}

void launch_setup_verify(const VerifySetup &p, cudaStream_t st) {
    setup_verify_kernel<<<p.batch * p.N, 128, 0, st>>>(p);
}

// Draft-pass rows (Algorithm 1 line 1; Section 3.2).  Block rows: slot 0 = E[root], slots 1..B-1 = mask
// embedding, position P + j.  Feature rows: target features of the positions committed last, whose K/V
// become head context at positions P - count .. P - 1 (or P .. P+count-1 while prefilling).
__global__ void __launch_bounds__(128) setup_draft_kernel(DraftSetup p) {
    const int R1 = p.batch * p.n_block;
    const int r = blockIdx.x + (p.features_only ? R1 : 0);
    const bf16 *src = nullptr;
    int s, pos, slot;
    if (r < R1) {
        s = r / p.B;
        const int j = r % p.B;
        const int P = p.seq_len[s];
        if (threadIdx.x == 0 && (P < 0 || P + p.B > p.capacity)) set_status(p.status, GLANCE_E_CAPACITY);
        pos = P + j;
        slot = P >= 0 ? P + j : -1;
        if (j == 0) {
            int t = p.root[s];
            if (t < 0 || t >= p.vocab) { t = 0; if (threadIdx.x == 0) set_status(p.status, GLANCE_E_BOUNDS); }
            src = p.embed + (size_t)t * p.out.H;
        } else {
            src = p.mask_embed;
        }
    } else {
        const int q = r - R1;
        s = q / p.FR;
        const int i = q % p.FR;
        const int P = p.seq_len[s];
        int cnt, base;
        if (p.feat_count) { cnt = p.feat_count[s]; base = P - cnt; }
        else { cnt = p.count_const; base = P; }
        if (cnt < 0 || cnt > p.FR || base < 0) { cnt = 0; if (threadIdx.x == 0) set_status(p.status, GLANCE_E_BOUNDS); }
        if (i < cnt) {
            pos = base + i;
            slot = base + i;
            src = p.feat + ((size_t)s * p.FR + i) * p.out.H;
        } else {
            pos = 0;
            slot = -1;
        }
    }
    if (threadIdx.x == 0) {
        p.meta.seq[r] = s;
        p.meta.pos[r] = pos;
        p.meta.kvrow[r] = kv_row_offset(p.geom, p.page_table, s, slot, p.status);
    }
    fill_rope_row(p.meta, r, pos, p.d, p.theta);
    emit_row(p.out, r, src, r < R1 ? p.gain_block : p.gain_feat);
}

void launch_setup_draft(const DraftSetup &p, cudaStream_t st) {
    const int R = (p.features_only ? 0 : p.batch * p.n_block) + p.batch * p.FR;
    setup_draft_kernel<<<R, 128, 0, st>>>(p);
}

// ------------------------------------------------------------------------------------------
// per-offset top-k and log-softmax (Assumption 1: marginals q_j over the full vocabulary), two stages.
// Stage 1: every warp owns 1024 consecutive vocabulary entries held in registers and emits its k best
// packed (value, id) keys (sorted) plus its max and sum of exponentials.  Stage 2: one warp per (sequence,
// offset) merges the warps' candidates and combines the partial log-sum-exp terms in a fixed order.  Both
// stages first find a threshold that the k best are known to reach (the k-th largest of the lane maxima / of
// the lists' heads), collect the few keys at or above it and rank only those.  Keys are unique, so the result
// does not depend on timing.
// ------------------------------------------------------------------------------------------
constexpr int kTopkWarpSpan = 1024;

__global__ void __launch_bounds__(128) topk_stage1_kernel(const float *logits, int B, int V, int k, int n_warps,
                                                          unsigned long long *cand, float *ml) {
    constexpr int CAP = 64;                              // candidates a warp may collect before it falls back
    __shared__ unsigned long long lists[4][CAP];
    const int L = B - 1;
    const int row = blockIdx.y;                         // (s, j-1)
    const int s = row / L, j = row % L + 1;
    const int wib = threadIdx.x >> 5;
    const int gw = blockIdx.x * 4 + wib;
    const int lane = threadIdx.x & 31;
    if (gw >= n_warps) return;
    const float *src = logits + ((size_t)s * B + j) * V;
    const int base = gw * kTopkWarpSpan;
    float val[32];
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const int c = base + i * 32 + lane;
        val[i] = c < V ? src[c] : -INFINITY;
        m = fmaxf(m, val[i]);
    }
    const float lane_max = m;
    m = warp_max(m);
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) sum += expf(val[i] - m);        // entries beyond V are -inf: they add exactly 0
    sum = warp_sum(sum);
    if (lane == 0) {
        ml[((size_t)row * n_warps + gw) * 2] = m;
        ml[((size_t)row * n_warps + gw) * 2 + 1] = sum;
    }
    unsigned long long *out = cand + ((size_t)row * n_warps + gw) * k;
    // Threshold: the k-th largest of the 32 lane maxima.  At least k values of the span are >= it, so every one of
    // the span's k best is; usually only a few more are.  (k <= 16 <= 32 lanes.)
    uint32_t cur = float_key(lane_max), thr = 0u;
    for (int t = 0; t < k; ++t) {
        thr = __reduce_max_sync(0xffffffffu, cur);
        const uint32_t holders = __ballot_sync(0xffffffffu, cur == thr);
        if (lane == __ffs(holders) - 1) cur = 0u;          // one holder leaves per round (0 sorts below every real value)
    }
    const float T = thr ? key_float(thr) : -INFINITY;    // fewer than k lanes hold anything: take everything
    // collect the packed keys of all values >= T
    unsigned long long *list = lists[wib];
    int count = 0;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const int c = base + i * 32 + lane;
        const bool hit = c < V && val[i] >= T;
        const uint32_t hits = __ballot_sync(0xffffffffu, hit);
        if (hits) {
            const int at = count + __popc(hits & ((1u << lane) - 1u));
            if (hit && at < CAP) list[at] = pack_val_id(val[i], c);
            count += __popc(hits);
        }
    }
    __syncwarp();
    if (count <= CAP) {
        // the k best of the few candidates (k rounds of a warp max over at most two keys per lane)
        unsigned long long c0 = lane < count ? list[lane] : 0ull, c1 = lane + 32 < count ? list[lane + 32] : 0ull;
        unsigned long long prev = ~0ull;
        for (int t = 0; t < k; ++t) {
            unsigned long long best = 0ull;
            if (c0 < prev && c0 > best) best = c0;
            if (c1 < prev && c1 > best) best = c1;
            best = warp_max_u64(best);
            if (lane == 0) out[t] = best;
            prev = best;
        }
        return;
    }
    // many equal values at the threshold (ties): exact selection over the whole span
    unsigned long long prev = ~0ull;
    for (int t = 0; t < k; ++t) {
        unsigned long long best = 0ull;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int c = base + i * 32 + lane;
            const unsigned long long key = c < V ? pack_val_id(val[i], c) : 0ull;
            if (key < prev && key > best) best = key;
        }
        best = warp_max_u64(best);
        if (lane == 0) out[t] = best;
        prev = best;
    }
}

// Stage 2: one warp per (sequence, offset).  The stage-1 lists are sorted, so the k-th largest of their heads is a
// threshold that all of the row's k best keys reach; the few keys at or above it are collected and ranked.
__global__ void __launch_bounds__(32) topk_stage2_kernel(int k, int n_warps, const unsigned long long *cand,
                                                         const float *ml, int32_t *ids, float *lp) {
    constexpr int CAP = 64;
    __shared__ unsigned long long list[CAP];
    const int row = blockIdx.x, lane = threadIdx.x;
    const float *rml = ml + (size_t)row * n_warps * 2;
    const unsigned long long *rc = cand + (size_t)row * n_warps * k;
    // log-sum-exp over the spans, fixed order: lane l adds spans l, l + 32, ...; lanes are then summed by shuffles
    float M = -INFINITY;
    for (int w = lane; w < n_warps; w += 32) M = fmaxf(M, rml[2 * w]);
    M = warp_max(M);
    float sum = 0.f;
    for (int w = lane; w < n_warps; w += 32) sum += rml[2 * w + 1] * expf(rml[2 * w] - M);
    sum = warp_sum(sum);
    const float lse = M + logf(sum);
    // threshold = k-th largest head (heads are unique keys); up to 8 heads per lane are held in registers
    unsigned long long thr = ~0ull;
    if (n_warps <= 256) {
        unsigned long long h0 = 0, h1 = 0, h2 = 0, h3 = 0, h4 = 0, h5 = 0, h6 = 0, h7 = 0;
        if (lane < n_warps) h0 = rc[(size_t)lane * k];
        if (lane + 32 < n_warps) h1 = rc[(size_t)(lane + 32) * k];
        if (lane + 64 < n_warps) h2 = rc[(size_t)(lane + 64) * k];
        if (lane + 96 < n_warps) h3 = rc[(size_t)(lane + 96) * k];
        if (lane + 128 < n_warps) h4 = rc[(size_t)(lane + 128) * k];
        if (lane + 160 < n_warps) h5 = rc[(size_t)(lane + 160) * k];
        if (lane + 192 < n_warps) h6 = rc[(size_t)(lane + 192) * k];
        if (lane + 224 < n_warps) h7 = rc[(size_t)(lane + 224) * k];
        for (int t = 0; t < k; ++t) {
            unsigned long long best = 0ull;
#define GLANCE_HEAD(h) if (h < thr && h > best) best = h;
            GLANCE_HEAD(h0) GLANCE_HEAD(h1) GLANCE_HEAD(h2) GLANCE_HEAD(h3) GLANCE_HEAD(h4) GLANCE_HEAD(h5) GLANCE_HEAD(h6) GLANCE_HEAD(h7)
#undef GLANCE_HEAD
            thr = warp_max_u64(best);
        }
    } else {
        for (int t = 0; t < k; ++t) {
            unsigned long long best = 0ull;
            for (int w = lane; w < n_warps; w += 32) {
                const unsigned long long h = rc[(size_t)w * k];
                if (h < thr && h > best) best = h;
            }
            thr = warp_max_u64(best);
        }
    }
    // every key >= thr (thr == 0: fewer than k spans hold anything -- then every non-empty key qualifies)
    const int n = n_warps * k;
    int count = 0;
    for (int c0 = 0; c0 < n; c0 += 128) {
        unsigned long long key4[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {                    // four independent loads in flight
            const int c = c0 + u * 32 + lane;
            key4[u] = c < n ? rc[c] : 0ull;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const bool hit = key4[u] != 0ull && key4[u] >= thr;
            const uint32_t hits = __ballot_sync(0xffffffffu, hit);
            if (hits) {
                const int at = count + __popc(hits & ((1u << lane) - 1u));
                if (hit && at < CAP) list[at] = key4[u];
                count += __popc(hits);
            }
        }
    }
    __syncwarp();
    unsigned long long prev = ~0ull;
    if (count <= CAP) {
        const unsigned long long a0 = lane < count ? list[lane] : 0ull, a1 = lane + 32 < count ? list[lane + 32] : 0ull;
        for (int t = 0; t < k; ++t) {
            unsigned long long best = 0ull;
            if (a0 < prev && a0 > best) best = a0;
            if (a1 < prev && a1 > best) best = a1;
            best = warp_max_u64(best);
            if (lane == 0) {
                ids[(size_t)row * k + t] = unpack_id(best);
                lp[(size_t)row * k + t] = unpack_val(best) - lse;
            }
            prev = best;
        }
        return;
    }
    for (int t = 0; t < k; ++t) {                        // (not reached with unique keys; kept for safety)
        unsigned long long best = 0ull;
        for (int c = lane; c < n; c += 32) {
            const unsigned long long key = rc[c];
            if (key < prev && key > best) best = key;
        }
        best = warp_max_u64(best);
        if (lane == 0) {
            ids[(size_t)row * k + t] = unpack_id(best);
            lp[(size_t)row * k + t] = unpack_val(best) - lse;
        }
        prev = best;
    }
}

int topk_warps(int V) { return (V + kTopkWarpSpan - 1) / kTopkWarpSpan; }

void launch_topk(const float *logits, int batch, int B, int V, int k, int32_t *ids, float *lp,
                 unsigned long long *cand, float *ml, cudaStream_t st) {
    if (B < 2) return;
    const int rows = batch * (B - 1), nw = topk_warps(V);
    dim3 g1((nw + 3) / 4, rows);
    topk_stage1_kernel<<<g1, 128, 0, st>>>(logits, B, V, k, nw, cand, ml);
    topk_stage2_kernel<<<rows, 32, 0, st>>>(k, nw, cand, ml, ids, lp);
}

// ------------------------------------------------------------------------------------------
// Merge of the draft LM head's per-tile shares (gemm_tc_kernel mode 5) into the per-offset top-k and log-softmax.
// One block per (sequence, offset).  The tiles left, for this row, (max, sum exp) and the keys that reached the
// row's bound at the time; the bound's final value (the smallest of the row's k class maxima) is what at least k
// entries of the row reach, so the k best are among the emitted keys at or above it.  Log-sum-exp: every thread folds the tiles t = tid, tid + 1024, ... in order,
// the threads' shares are then added in a fixed tree (bit-reproducible).  The keys at or above the final bound
// (few) are collected into shared memory in any order and ranked by one warp; keys are unique, so the ranking does
// not depend on the order of collection.  The row's bound is re-armed (0) for the next launch.
// ------------------------------------------------------------------------------------------
constexpr int kMergeThreads = 1024;
constexpr int kMergeCap = 512;                           // keys a row may collect before it falls back to full scans

__global__ void __launch_bounds__(kMergeThreads) topk_merge_kernel(int B, int R, int tiles, int k, uint32_t *thr,
                                                                   const float *ml, const int32_t *cnt,
                                                                   const unsigned long long *cand, int32_t *ids, float *lp) {
    static_assert(kMergeThreads == 1024, "the second reduction level takes exactly 32 warps");
    __shared__ float red_m[32], red_s[32];
    __shared__ unsigned long long list[kMergeCap];
    __shared__ int n_list;
    __shared__ unsigned long long best_w[kMergeThreads / 32];
    const int L = B - 1;
    const int out_row = blockIdx.x;                      // (s, j-1)
    const int s = out_row / L, j = out_row % L + 1;
    const int r = s * B + j;                             // row of the LM-head launch
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    tc::pdl_wait();                                      // launched early; everything it reads is the LM head's output
    // ---- log-sum-exp over the tiles
    float M = -INFINITY, S = 0.f;
    for (int t = tid; t < tiles; t += kMergeThreads) {
        const float m = __ldcg(ml + 2 * ((size_t)t * R + r)), e = __ldcg(ml + 2 * ((size_t)t * R + r) + 1);
        const float nm = fmaxf(M, m);
        S = (M == -INFINITY ? 0.f : S * expf(M - nm)) + (m == -INFINITY ? 0.f : e * expf(m - nm));
        M = nm;
    }
    // fixed tree: lanes by shuffles, then the 32 warps' shares by the first warp
    auto fold = [](float &m0, float &s0, float m1, float s1) {
        const float nm = fmaxf(m0, m1);
        s0 = (m0 == -INFINITY ? 0.f : s0 * expf(m0 - nm)) + (m1 == -INFINITY ? 0.f : s1 * expf(m1 - nm));
        m0 = nm;
    };
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) fold(M, S, __shfl_xor_sync(0xffffffffu, M, o), __shfl_xor_sync(0xffffffffu, S, o));
    if (lane == 0) { red_m[wid] = M; red_s[wid] = S; }
    if (tid == 0) n_list = 0;
    __syncthreads();
    if (wid == 0) {
        M = red_m[lane];
        S = red_s[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) fold(M, S, __shfl_xor_sync(0xffffffffu, M, o), __shfl_xor_sync(0xffffffffu, S, o));
        if (lane == 0) { red_m[0] = M; red_s[0] = S; }
    }
    __syncthreads();
    const float lse = red_m[0] + logf(red_s[0]);
    // ---- the keys at or above the row's final bound
    uint32_t T = 0xffffffffu;                            // the smallest of the row's k class maxima (0: a class stayed empty)
    for (int b = 0; b < k; ++b) T = min(T, __ldcg(thr + (size_t)r * kTopkTileCap + b));
    // one thread per (tile, key slot): the count and the key are fetched independently (a slot beyond the tile's count
    // holds an older launch's key and is ignored), so the loads of a thread's few iterations are all in flight together
    for (int idx0 = tid; idx0 < tiles * kTopkTileCap; idx0 += 8 * kMergeThreads) {
        int c8[8];
        unsigned long long key8[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {                    // eight independent (count, key) pairs in flight
            const int idx = idx0 + u * kMergeThreads;
            c8[u] = 0;
            key8[u] = 0ull;
            if (idx < tiles * kTopkTileCap) {
                const size_t slot = (size_t)(idx / kTopkTileCap) * R + r;
                c8[u] = __ldcg(cnt + slot);
                key8[u] = __ldcg(cand + slot * kTopkTileCap + idx % kTopkTileCap);
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = (idx0 + u * kMergeThreads) % kTopkTileCap;
            if (i < c8[u] && (uint32_t)(key8[u] >> 32) >= T) {
                const int at = atomicAdd(&n_list, 1);
                if (at < kMergeCap) list[at] = key8[u];
            }
        }
    }
    __syncthreads();
    const int n = n_list;
    unsigned long long prev = ~0ull;
    if (n <= kMergeCap) {
        if (wid == 0) {
            for (int t = 0; t < k; ++t) {
                unsigned long long best = 0ull;
                for (int c = lane; c < n; c += 32) {
                    const unsigned long long key = list[c];
                    if (key < prev && key > best) best = key;
                }
                best = warp_max_u64(best);
                if (lane == 0) {
                    ids[(size_t)out_row * k + t] = unpack_id(best);
                    lp[(size_t)out_row * k + t] = unpack_val(best) - lse;
                }
                prev = best;
            }
        }
    } else {
        // very many equal values at the bound: k full scans over the emitted keys
        for (int t = 0; t < k; ++t) {
            unsigned long long best = 0ull;
            for (int tl = tid; tl < tiles; tl += kMergeThreads) {
                const size_t slot = (size_t)tl * R + r;
                const int c = __ldcg(cnt + slot);
                for (int i = 0; i < c; ++i) {
                    const unsigned long long key = __ldcg(cand + slot * kTopkTileCap + i);
                    if (key < prev && key > best) best = key;
                }
            }
            best = warp_max_u64(best);
            if (lane == 0) best_w[wid] = best;
            __syncthreads();
            best = 0ull;
            for (int w = 0; w < kMergeThreads / 32; ++w) best = best_w[w] > best ? best_w[w] : best;
            if (tid == 0) {
                ids[(size_t)out_row * k + t] = unpack_id(best);
                lp[(size_t)out_row * k + t] = unpack_val(best) - lse;
            }
            prev = best;
            __syncthreads();
        }
    }
    if (tid < kTopkTileCap) thr[(size_t)r * kTopkTileCap + tid] = 0u;   // every read of the bounds is behind the barrier above
}

void launch_topk_merge(int batch, int B, int tiles, int k, uint32_t *thr, const float *ml, const int32_t *cnt,
                       const unsigned long long *cand, int32_t *ids, float *lp, cudaStream_t st) {
    if (B < 2) return;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(batch * (B - 1), 1, 1);
    cfg.blockDim = dim3(kMergeThreads, 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // its blocks are placed while the LM head drains
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, topk_merge_kernel, B, batch * B, tiles, k, thr, (const float *)ml, (const int32_t *)cnt,
                       (const unsigned long long *)cand, ids, lp);
}

__global__ void prefill_advance_kernel(int32_t *seq_len, int32_t *root, int32_t *feat_count, const int32_t *argmax,
                                       int count) {
    if (threadIdx.x == 0) {
        seq_len[0] += count;
        if (argmax) root[0] = argmax[count - 1];
        feat_count[0] = 0;
    }
}

void launch_prefill_advance(int32_t *seq_len, int32_t *root, int32_t *feat_count, const int32_t *argmax, int count,
                            cudaStream_t st) {
    prefill_advance_kernel<<<1, 32, 0, st>>>(seq_len, root, feat_count, argmax, count);
}

}  // namespace glance
