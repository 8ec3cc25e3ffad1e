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
__global__ void __launch_bounds__(256) norm_kernel(float *x, const float *part, int S, size_t split_stride, int ldp,
                                                   int H, const bf16 *gain_a, const bf16 *gain_b, int split_row,
                                                   float eps, bf16 *xn, bf16 *hidden_out) {
    extern __shared__ float row[];
    __shared__ float red[8];
    const int r = blockIdx.x;
    float *xr = x + (size_t)r * H;
    float ss = 0.f;
    for (int c = threadIdx.x; c < H; c += blockDim.x) {
        float v = xr[c];
        for (int s = 0; s < S; ++s) v += part[s * split_stride + (size_t)r * ldp + c];
        row[c] = v;
        ss += v * v;
        if (S > 0) xr[c] = v;
        if (hidden_out) hidden_out[(size_t)r * H + c] = __float2bfloat16(v);
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    const float inv = rsqrtf(tot / (float)H + eps);
    const bf16 *g = (r >= split_row) ? gain_b : gain_a;
    if (xn)
        for (int c = threadIdx.x; c < H; c += blockDim.x)
            xn[(size_t)r * H + c] = __float2bfloat16(row[c] * inv * __bfloat162float(g[c]));
}

void launch_norm(float *x, const float *part, int S, size_t part_split_stride, int ldp, int R, int H,
                 const bf16 *gain_a, const bf16 *gain_b, int split_row, float eps, bf16 *xn, bf16 *hidden_out,
                 cudaStream_t st) {
    norm_kernel<<<R, 256, H * sizeof(float), st>>>(x, part, S, part_split_stride, ldp, H, gain_a,
                                                   gain_b ? gain_b : gain_a, split_row, eps, xn, hidden_out);
}

// ------------------------------------------------------------------------------------------
// QKV split-K reduction + rotary (pairs (i, i + d/2)) + paged K/V write
// ------------------------------------------------------------------------------------------
__global__ void rope_kv_kernel(RopeKv p) {
    const int r = blockIdx.x;
    const int half = p.d >> 1;
    const int slot_pos = p.meta.kvslot[r];
    const int s = p.meta.seq[r];
    const float *cs = p.meta.rope_cos + (size_t)r * half;
    const float *sn = p.meta.rope_sin + (size_t)r * half;
    const int n_rot = (p.Hq + p.Hkv) * half;       // rotated pairs (q heads then k heads)
    const int n_v = p.Hkv * p.d;
    bf16 *krow = nullptr, *vrow = nullptr;
    if (slot_pos >= 0) {
        const int pg = slot_pos / kPage;
        bool ok = pg < p.geom.max_pages_per_seq;
        int page = ok ? p.page_table[(size_t)s * p.geom.max_pages_per_seq + pg] : 0;
        if (page < 0 || page >= p.geom.n_pages) ok = false;
        if (ok) {
            krow = p.pool_layer + p.geom.row(page, 0, 0, slot_pos % kPage);
            vrow = p.pool_layer + p.geom.row(page, 1, 0, slot_pos % kPage);
        } else if (threadIdx.x == 0) {
            set_status(p.status, GLANCE_E_BOUNDS);
        }
    }
    const size_t head_stride = (size_t)kPage * p.d;    // distance between kv heads of one (page, kv)
    for (int e = threadIdx.x; e < n_rot + n_v; e += blockDim.x) {
        if (e < n_rot) {
            const int h = e / half, i = e % half;
            if (h < p.Hq && r >= p.Rq) continue;
            const int col = h * p.d + i;
            float a = 0.f, b = 0.f;
            for (int sp = 0; sp < p.S; ++sp) {
                const float *y = p.part + sp * p.split_stride + (size_t)r * p.ldy;
                a += y[col];
                b += y[col + half];
            }
            const float c = cs[i], sv = sn[i];
            const float ra = a * c - b * sv, rb = b * c + a * sv;
            if (h < p.Hq) {
                bf16 *q = p.q + (size_t)r * p.Hq * p.d + col;
                q[0] = __float2bfloat16(ra);
                q[half] = __float2bfloat16(rb);
            } else if (krow) {
                bf16 *k = krow + (size_t)(h - p.Hq) * head_stride + i;
                k[0] = __float2bfloat16(ra);
                k[half] = __float2bfloat16(rb);
            }
        } else if (vrow) {
            const int ev = e - n_rot;
            const int h = ev / p.d, i = ev % p.d;
            const int col = (p.Hq + p.Hkv) * p.d + ev;
            float a = 0.f;
            for (int sp = 0; sp < p.S; ++sp) a += p.part[sp * p.split_stride + (size_t)r * p.ldy + col];
            vrow[(size_t)h * head_stride + i] = __float2bfloat16(a);
        }
    }
}

void launch_rope_kv(const RopeKv &p, cudaStream_t st) { rope_kv_kernel<<<p.R, 256, 0, st>>>(p); }

// ------------------------------------------------------------------------------------------
// SwiGLU: act = silu(gate) * up
// ------------------------------------------------------------------------------------------
__global__ void swiglu_kernel(const float *part, int ldp, int F, bf16 *act) {
    const int r = blockIdx.y;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= F) return;
    const float g = part[(size_t)r * ldp + c], u = part[(size_t)r * ldp + F + c];
    act[(size_t)r * F + c] = __float2bfloat16(g / (1.f + __expf(-g)) * u);
}

void launch_swiglu(const float *part, int ldp, int R, int F, bf16 *act, cudaStream_t st) {
    dim3 grid((F + 255) / 256, R);
    swiglu_kernel<<<grid, 256, 0, st>>>(part, ldp, F, act);
}

// ------------------------------------------------------------------------------------------
// argmax over the vocabulary (value desc, id asc) on fp32 logits
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

__global__ void __launch_bounds__(512) argmax_kernel(const float *logits, int V, int32_t *out) {
    __shared__ unsigned long long sh[16];
    const float *row = logits + (size_t)blockIdx.x * V;
    unsigned long long best = 0;
    for (int c = threadIdx.x; c < V; c += blockDim.x) {
        unsigned long long k = pack_val_id(row[c], c);
        best = k > best ? k : best;
    }
    best = block_max_u64(best, sh);
    if (threadIdx.x == 0) out[blockIdx.x] = unpack_id(best);
}

void launch_argmax(const float *logits, int R, int V, int32_t *out, cudaStream_t st) {
    argmax_kernel<<<R, 512, 0, st>>>(logits, V, out);
}

// ------------------------------------------------------------------------------------------
// per-offset top-k and log-softmax (Assumption 1: marginals q_j over the full vocabulary)
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512) topk_kernel(const float *logits, int B, int V, int k, int32_t *ids, float *lp) {
    __shared__ unsigned long long sh[16];
    __shared__ float shf[16];
    const int L = B - 1;
    const int s = blockIdx.x / L, j = blockIdx.x % L + 1;
    const float *row = logits + ((size_t)s * B + j) * V;
    // max
    float m = -INFINITY;
    for (int c = threadIdx.x; c < V; c += blockDim.x) m = fmaxf(m, row[c]);
    m = warp_max(m);
    if ((threadIdx.x & 31) == 0) shf[threadIdx.x >> 5] = m;
    __syncthreads();
    m = shf[0];
    for (int w = 1; w < (blockDim.x >> 5); ++w) m = fmaxf(m, shf[w]);
    __syncthreads();
    // sum exp
    float sum = 0.f;
    for (int c = threadIdx.x; c < V; c += blockDim.x) sum += expf(row[c] - m);
    sum = warp_sum(sum);
    if ((threadIdx.x & 31) == 0) shf[threadIdx.x >> 5] = sum;
    __syncthreads();
    sum = 0.f;
    for (int w = 0; w < (blockDim.x >> 5); ++w) sum += shf[w];
    const float lse = m + logf(sum);
    // k rounds of "largest key strictly below the previous winner"
    unsigned long long prev = ~0ull;
    for (int t = 0; t < k; ++t) {
        unsigned long long best = 0;
        for (int c = threadIdx.x; c < V; c += blockDim.x) {
            unsigned long long key = pack_val_id(row[c], c);
            if (key < prev && key > best) best = key;
        }
        best = block_max_u64(best, sh);
        if (threadIdx.x == 0) {
            ids[((size_t)s * L + (j - 1)) * k + t] = unpack_id(best);
            lp[((size_t)s * L + (j - 1)) * k + t] = unpack_val(best) - lse;
        }
        prev = best;
    }
}

void launch_topk(const float *logits, int batch, int B, int V, int k, int32_t *ids, float *lp, cudaStream_t st) {
    if (B < 2) return;
    topk_kernel<<<batch * (B - 1), 512, 0, st>>>(logits, B, V, k, ids, lp);
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
