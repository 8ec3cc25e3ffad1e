// Row setup, normalisation, rotary + paged K/V write, SwiGLU, argmax and top-k kernels of the round.
#include "kernels.cuh"

namespace glance {

// ------------------------------------------------------------------------------------------
// rotary table of one row: angle = pos * theta^(-2i/d), evaluated in double (one row per block)
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void fill_rope_row(const RowMeta &m, int r, int pos, int d, float theta) {
    const int half = d >> 1;
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        double inv = pow((double)theta, -(2.0 * i) / (double)d);
        double s, c;
        sincos((double)pos * inv, &s, &c);
        m.rope_cos[(size_t)r * half + i] = (float)c;
        m.rope_sin[(size_t)r * half + i] = (float)s;
    }
}

// Verify-pass rows (Algorithm 1 line 3: pack the root and the tree).  Row r = s*N + i is node i of
// sequence s at rotary position P + depth[i]; its K/V go to cache row P + i.  In prefill mode the rows are
// a causal chain of `count` given embeddings / token ids and the chain's ancestor mask is emitted.
__global__ void setup_verify_kernel(VerifySetup p) {
    const int r = blockIdx.x;
    const int s = r / p.N, i = r % p.N;
    const int P = p.seq_len[s];
    const bool prefill = (p.token == nullptr);
    int depth = prefill ? i : p.depth[r];
    if (!prefill && (depth < 0 || depth > kMaxBlock)) depth = 0;
    if (threadIdx.x == 0) {
        if (P < 0 || P + p.N > p.capacity) set_status(p.status, GLANCE_E_CAPACITY);
        p.meta.seq[r] = s;
        p.meta.pos[r] = P + depth;
        p.meta.kvslot[r] = P + i;
    }
    fill_rope_row(p.meta, r, P + depth, p.d, p.theta);
    float *x = p.x + (size_t)r * p.H;
    const bf16 *src = nullptr;
    if (prefill) {
        if (i < p.count) {
            if (p.row_embeds) src = p.row_embeds + (size_t)i * p.H;
            else {
                int t = p.row_ids[i];
                if (t < 0 || t >= p.vocab) { t = 0; if (threadIdx.x == 0) set_status(p.status, GLANCE_E_BOUNDS); }
                src = p.embed + (size_t)t * p.H;
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
        src = p.embed + (size_t)t * p.H;
    }
    for (int c = threadIdx.x; c < p.H; c += blockDim.x) x[c] = src ? __bfloat162float(src[c]) : 0.f;
}

void launch_setup_verify(const VerifySetup &p, cudaStream_t st) {
    setup_verify_kernel<<<p.batch * p.N, 128, 0, st>>>(p);
}

// Draft-pass rows (Algorithm 1 line 1; Section 3.2).  Block rows: slot 0 = E[root], slots 1..B-1 = mask
// embedding, position P + j.  Feature rows: target features of the positions committed last, whose K/V
// become head context at positions P - count .. P - 1 (or P .. P+count-1 while prefilling).
__global__ void setup_draft_kernel(DraftSetup p) {
    const int r = blockIdx.x;
    const int R1 = p.batch * p.n_block;
    float *x = p.x + (size_t)r * p.H;
    const bf16 *src = nullptr;
    int s, pos, slot;
    if (r < R1) {
        s = r / p.B;
        const int j = r % p.B;
        const int P = p.seq_len[s];
        if (threadIdx.x == 0 && (P < 0 || P + p.B > p.capacity)) set_status(p.status, GLANCE_E_CAPACITY);
        pos = P + j;
        slot = P + j;
        if (j == 0) {
            int t = p.root[s];
            if (t < 0 || t >= p.vocab) { t = 0; if (threadIdx.x == 0) set_status(p.status, GLANCE_E_BOUNDS); }
            src = p.embed + (size_t)t * p.H;
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
            src = p.feat + ((size_t)s * p.FR + i) * p.H;
        } else {
            pos = 0;
            slot = -1;
        }
    }
    if (threadIdx.x == 0) {
        p.meta.seq[r] = s;
        p.meta.pos[r] = pos;
        p.meta.kvslot[r] = slot;
    }
    fill_rope_row(p.meta, r, pos, p.d, p.theta);
    for (int c = threadIdx.x; c < p.H; c += blockDim.x) x[c] = src ? __bfloat162float(src[c]) : 0.f;
}

void launch_setup_draft(const DraftSetup &p, cudaStream_t st) {
    const int R = p.batch * p.n_block + p.batch * p.FR;
    setup_draft_kernel<<<R, 128, 0, st>>>(p);
}

// ------------------------------------------------------------------------------------------
// residual add (split-K partials, fixed order) + RMSNorm -> bf16
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) norm_kernel(float *x, const float *part, int S, size_t split_stride, int ldp,
                                                    int H, const bf16 *gain_a, const bf16 *gain_b, int split_row,
                                                    float eps, bf16 *xn, bf16 *hidden_out) {
    extern __shared__ float4 row4[];
    __shared__ float red[32];
    const int r = blockIdx.x;
    const int H4 = H >> 2;
    float4 *xr = reinterpret_cast<float4 *>(x + (size_t)r * H);
    float ss = 0.f;
    for (int c = threadIdx.x; c < H4; c += blockDim.x) {
        float4 v = xr[c];
        for (int s = 0; s < S; ++s) {
            const float4 p = __ldcg(reinterpret_cast<const float4 *>(part + s * split_stride + (size_t)r * ldp) + c);
            v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
        }
        row4[c] = v;
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        if (S > 0) xr[c] = v;
        if (hidden_out) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
            uint2 o;
            o.x = *reinterpret_cast<uint32_t *>(&lo);
            o.y = *reinterpret_cast<uint32_t *>(&hi);
            reinterpret_cast<uint2 *>(hidden_out + (size_t)r * H)[c] = o;
        }
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    const int nw = (blockDim.x + 31) >> 5;
    for (int w = 0; w < nw; ++w) tot += red[w];
    const float inv = rsqrtf(tot / (float)H + eps);
    const bf16 *g = (r >= split_row) ? gain_b : gain_a;
    if (xn)
        for (int c = threadIdx.x; c < H4; c += blockDim.x) {
            const float4 v = row4[c];
            const uint2 gg = reinterpret_cast<const uint2 *>(g)[c];
            const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162 *>(&gg.x);
            const __nv_bfloat162 g23 = *reinterpret_cast<const __nv_bfloat162 *>(&gg.y);
            __nv_bfloat162 lo = __floats2bfloat162_rn(v.x * inv * __low2float(g01), v.y * inv * __high2float(g01));
            __nv_bfloat162 hi = __floats2bfloat162_rn(v.z * inv * __low2float(g23), v.w * inv * __high2float(g23));
            uint2 o;
            o.x = *reinterpret_cast<uint32_t *>(&lo);
            o.y = *reinterpret_cast<uint32_t *>(&hi);
            reinterpret_cast<uint2 *>(xn + (size_t)r * H)[c] = o;
        }
}

void launch_norm(float *x, const float *part, int S, size_t part_split_stride, int ldp, int R, int H,
                 const bf16 *gain_a, const bf16 *gain_b, int split_row, float eps, bf16 *xn, bf16 *hidden_out,
                 cudaStream_t st) {
    int threads = ((H / 4) + 31) / 32 * 32;
    threads = threads > 1024 ? 1024 : threads;
    norm_kernel<<<R, threads, H * sizeof(float), st>>>(x, part, S, part_split_stride, ldp, H, gain_a,
                                                       gain_b ? gain_b : gain_a, split_row, eps, xn, hidden_out);
}

// ------------------------------------------------------------------------------------------
// QKV split-K reduction + rotary (pairs (i, i + d/2)) + paged K/V write
// ------------------------------------------------------------------------------------------
__global__ void rope_kv_kernel(RopeKv p) {
    // grid (R, Hq + 2 Hkv): one block per (row, head); heads are ordered q..., k..., v...
    const int r = blockIdx.x, h = blockIdx.y;
    const int half = p.d >> 1;
    const bool is_q = h < p.Hq, is_k = !is_q && h < p.Hq + p.Hkv;
    if (is_q && r >= p.Rq) return;
    const int slot_pos = p.meta.kvslot[r];
    bf16 *dst = nullptr;
    if (is_q) {
        dst = p.q + ((size_t)r * p.Hq + h) * p.d;
    } else {
        if (slot_pos < 0) return;
        const int s = p.meta.seq[r];
        const int pg = slot_pos / kPage;
        bool ok = pg < p.geom.max_pages_per_seq;
        int page = ok ? p.page_table[(size_t)s * p.geom.max_pages_per_seq + pg] : 0;
        if (page < 0 || page >= p.geom.n_pages) ok = false;
        if (!ok) {
            if (threadIdx.x == 0) set_status(p.status, GLANCE_E_BOUNDS);
            return;
        }
        const int kvh = is_k ? h - p.Hq : h - p.Hq - p.Hkv;
        dst = p.pool_layer + p.geom.row(page, is_k ? 0 : 1, kvh, slot_pos % kPage);
    }
    const int col0 = h * p.d;
    const float *y = p.part + (size_t)r * p.ldy + col0;
    if (is_q || is_k) {
        const float *cs = p.meta.rope_cos + (size_t)r * half;
        const float *sn = p.meta.rope_sin + (size_t)r * half;
        for (int i = threadIdx.x; i < half; i += blockDim.x) {
            float a = 0.f, b = 0.f;
            for (int sp = 0; sp < p.S; ++sp) {
                a += __ldcg(y + sp * p.split_stride + i);
                b += __ldcg(y + sp * p.split_stride + i + half);
            }
            const float c = cs[i], sv = sn[i];
            dst[i] = __float2bfloat16(a * c - b * sv);
            dst[i + half] = __float2bfloat16(b * c + a * sv);
        }
    } else {
        for (int i = threadIdx.x; i < p.d; i += blockDim.x) {
            float a = 0.f;
            for (int sp = 0; sp < p.S; ++sp) a += __ldcg(y + sp * p.split_stride + i);
            dst[i] = __float2bfloat16(a);
        }
    }
}

void launch_rope_kv(const RopeKv &p, cudaStream_t st) {
    dim3 grid(p.R, p.Hq + 2 * p.Hkv);
    rope_kv_kernel<<<grid, 64, 0, st>>>(p);
}

// ------------------------------------------------------------------------------------------
// block-wide max of packed (value desc, id asc) keys
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long block_max_u64(unsigned long long v, unsigned long long *sh) {
    v = warp_max_u64(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    unsigned long long r = 0;
    const int nw = blockDim.x >> 5;
    for (int w = 0; w < nw; ++w) r = sh[w] > r ? sh[w] : r;
    return r;
}

// ------------------------------------------------------------------------------------------
// per-offset top-k and log-softmax (Assumption 1: marginals q_j over the full vocabulary), two stages.
// Stage 1: every warp owns 1024 consecutive vocabulary entries held in registers and emits its k best
// packed (value, id) keys plus its max and sum of exponentials.  Stage 2: one block per (sequence,
// offset) merges the warps' candidates with k rounds of a block-wide max and combines the partial
// log-sum-exp terms in a fixed order.  Keys are unique, so the result does not depend on timing.
// ------------------------------------------------------------------------------------------
constexpr int kTopkWarpSpan = 1024;

__global__ void __launch_bounds__(128) topk_stage1_kernel(const float *logits, int B, int V, int k, int n_warps,
                                                          unsigned long long *cand, float *ml) {
    const int L = B - 1;
    const int row = blockIdx.y;                         // (s, j-1)
    const int s = row / L, j = row % L + 1;
    const int gw = blockIdx.x * 4 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (gw >= n_warps) return;
    const float *src = logits + ((size_t)s * B + j) * V;
    const int base = gw * kTopkWarpSpan;
    unsigned long long key[32];
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const int c = base + i * 32 + lane;
        const float v = c < V ? src[c] : -INFINITY;
        key[i] = c < V ? pack_val_id(v, c) : 0ull;
        m = fmaxf(m, v);
    }
    m = warp_max(m);
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const int c = base + i * 32 + lane;
        if (c < V) sum += expf(unpack_val(key[i]) - m);
    }
    sum = warp_sum(sum);
    if (lane == 0) {
        ml[((size_t)row * n_warps + gw) * 2] = m;
        ml[((size_t)row * n_warps + gw) * 2 + 1] = sum;
    }
    unsigned long long prev = ~0ull;
    for (int t = 0; t < k; ++t) {
        unsigned long long best = 0ull;
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (key[i] < prev && key[i] > best) best = key[i];
        best = warp_max_u64(best);
        if (lane == 0) cand[((size_t)row * n_warps + gw) * k + t] = best;
        prev = best;
    }
}

__global__ void __launch_bounds__(256) topk_stage2_kernel(int k, int n_warps, const unsigned long long *cand,
                                                          const float *ml, int32_t *ids, float *lp) {
    __shared__ unsigned long long sh[16];
    __shared__ float shf[16];
    const int row = blockIdx.x;
    const float *rml = ml + (size_t)row * n_warps * 2;
    float M = -INFINITY;
    for (int w = threadIdx.x; w < n_warps; w += blockDim.x) M = fmaxf(M, rml[2 * w]);
    M = warp_max(M);
    if ((threadIdx.x & 31) == 0) shf[threadIdx.x >> 5] = M;
    __syncthreads();
    M = shf[0];
    for (int w = 1; w < 8; ++w) M = fmaxf(M, shf[w]);
    __syncthreads();
    // fixed-order sum: thread t adds warps t, t+256, ...; partial sums are then added in warp/lane order
    float sum = 0.f;
    for (int w = threadIdx.x; w < n_warps; w += blockDim.x) sum += rml[2 * w + 1] * expf(rml[2 * w] - M);
    sum = warp_sum(sum);
    if ((threadIdx.x & 31) == 0) shf[threadIdx.x >> 5] = sum;
    __syncthreads();
    sum = 0.f;
    for (int w = 0; w < 8; ++w) sum += shf[w];
    const float lse = M + logf(sum);
    const unsigned long long *rc = cand + (size_t)row * n_warps * k;
    const int n = n_warps * k;
    unsigned long long prev = ~0ull;
    for (int t = 0; t < k; ++t) {
        unsigned long long best = 0ull;
        for (int c = threadIdx.x; c < n; c += blockDim.x) {
            const unsigned long long key = rc[c];
            if (key < prev && key > best) best = key;
        }
        best = block_max_u64(best, sh);
        if (threadIdx.x == 0) {
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
    topk_stage2_kernel<<<rows, 256, 0, st>>>(k, nw, cand, ml, ids, lp);
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
