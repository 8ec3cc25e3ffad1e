// Split-KV paged attention of the packed tree rows (Definition 1: ancestor-masked target pass) and of
// the draft block (Section 3.2: every block slot sees the whole context and the whole block).
//
// One CTA = (64 packed query rows of one kv head, one key split).  The G query heads that share a kv
// head are packed into the row dimension (packed row = node * G + g), so each K/V page is fetched once
// per CTA for all of them.  Keys 0..P-1 (committed context) are always visible; key P + j is visible to
// the row of node i iff bit j of anc[i] is set (or always, when no mask is given).  One 64-key tile is
// exactly one KV page.  Scores and softmax are fp32 (online softmax in base 2), products on bf16
// tensor-core MMAs.  Splits are merged by the last CTA to arrive (no CTA waits on another).
#include "kernels.cuh"

namespace glance {

namespace {

constexpr int QT = 64;          // packed query rows per CTA (4 warps x 16)
constexpr int KT = kPage;       // keys per tile

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// byte offset of 16-byte chunk `c` of row `r` in a tile whose rows hold D bf16 (XOR swizzle within groups of 8 chunks)
template <int D>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
    return (uint32_t)(r * (D * 2) + (((c & ~7) | ((c ^ r) & 7)) << 4));
}

template <int D>
__global__ void __launch_bounds__(128) attn_kernel(AttnParams p) {
    constexpr int CH = D / 8;                  // 16-byte chunks per row
    constexpr int KS = D / 16;                 // k-steps of QK^T
    constexpr int DN = D / 8;                  // n-tiles of the output
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *sQ = smem;                                  // QT x D
    unsigned char *sK = sQ + QT * D * 2;                       // 2 x KT x D
    unsigned char *sV = sK + 2 * KT * D * 2;                   // 2 x KT x D
    float *sW = reinterpret_cast<float *>(sV + 2 * KT * D * 2);  // combine weights QT x S (S <= 32)
    __shared__ int sh_last;

    const int G = p.Hq / p.Hkv;
    const int PR = p.T * G;
    const int qt = blockIdx.x, kvh = blockIdx.y;
    const int s = blockIdx.z / p.S, split = blockIdx.z % p.S;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g8 = lane >> 2, t4 = lane & 3;

    const int P = p.seq_len[s];
    const int n_keys = P + p.T;
    const int n_tiles = (n_keys + KT - 1) / KT;
    const int t_begin = (int)((long long)split * n_tiles / p.S);
    const int t_end = (int)((long long)(split + 1) * n_tiles / p.S);
    const int32_t *pt = p.page_table + (size_t)s * p.geom.max_pages_per_seq;

    // ---- Q tile -> smem
    for (int it = tid; it < QT * CH; it += 128) {
        const int r = it / CH, c = it % CH;
        int pr = qt * QT + r;
        if (pr >= PR) pr = PR - 1;
        const int node = pr / G, g = pr % G;
        const bf16 *src = p.q + ((size_t)(s * p.T + node) * p.Hq + kvh * G + g) * D + c * 8;
        cp_async16(smem_u32(sQ + tile_off<D>(r, c)), src);
    }
    cp_async_commit();

    auto load_tile = [&](int t, int buf) {
        bool ok = t < p.geom.max_pages_per_seq;
        int page = ok ? pt[t] : 0;
        if (page < 0 || page >= p.geom.n_pages) ok = false;
        const bf16 *kbase = p.pool_layer + p.geom.row(ok ? page : 0, 0, kvh, 0);
        const bf16 *vbase = p.pool_layer + p.geom.row(ok ? page : 0, 1, kvh, 0);
        unsigned char *dK = sK + buf * KT * D * 2, *dV = sV + buf * KT * D * 2;
        const int valid = ok ? min(KT, n_keys - t * KT) : 0;
        for (int it = tid; it < KT * CH; it += 128) {
            const int r = it / CH, c = it % CH;
            if (r < valid) {
                cp_async16(smem_u32(dK + tile_off<D>(r, c)), kbase + (size_t)r * D + c * 8);
                cp_async16(smem_u32(dV + tile_off<D>(r, c)), vbase + (size_t)r * D + c * 8);
            } else {
                // rows beyond the last key may hold anything (NaN bits included): zero them
                *reinterpret_cast<int4 *>(dK + tile_off<D>(r, c)) = make_int4(0, 0, 0, 0);
                *reinterpret_cast<int4 *>(dV + tile_off<D>(r, c)) = make_int4(0, 0, 0, 0);
            }
        }
        if (!ok && tid == 0) set_status(p.status, GLANCE_E_BOUNDS);
    };

    if (t_begin < t_end) load_tile(t_begin, 0);
    cp_async_commit();

    // ---- per-thread rows: two rows (g8, g8+8) of this warp's 16
    int node_r[2];
    uint64_t anc_r[2][2] = {{0, 0}, {0, 0}};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        int pr = qt * QT + warp * 16 + g8 + 8 * h;
        if (pr >= PR) pr = PR - 1;
        node_r[h] = pr / G;
        if (p.anc) {
            const uint64_t *a = p.anc + ((size_t)s * p.T + node_r[h]) * p.W;
            anc_r[h][0] = a[0];
            anc_r[h][1] = p.W > 1 ? a[1] : 0ull;
        }
    }

    cp_async_wait<1>();          // Q landed
    __syncthreads();
    uint32_t qf[KS][4];
#pragma unroll
    for (int kk = 0; kk < KS; ++kk)
        ldsm_x4(smem_u32(sQ + tile_off<D>(warp * 16 + (lane & 15), kk * 2 + (lane >> 4))), qf[kk][0], qf[kk][1],
                qf[kk][2], qf[kk][3]);

    float o[DN][4];
#pragma unroll
    for (int j = 0; j < DN; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
    float m_r[2] = {-INFINITY, -INFINITY}, l_r[2] = {0.f, 0.f};
    const float sl2 = rsqrtf((float)D) * 1.4426950408889634f;

    for (int t = t_begin; t < t_end; ++t) {
        const int buf = (t - t_begin) & 1;
        if (t + 1 < t_end) load_tile(t + 1, buf ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const unsigned char *cK = sK + buf * KT * D * 2, *cV = sV + buf * KT * D * 2;

        // S = Q K^T : 8 n-tiles of 8 keys
        float sc[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f;
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) {
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                uint32_t b0, b1, b2, b3;
                const int mtx = lane >> 3;
                ldsm_x4(smem_u32(cK + tile_off<D>(j * 8 + (lane & 7) + (mtx >> 1) * 8, kk * 2 + (mtx & 1))), b0, b1, b2, b3);
                mma_bf16(sc[j], qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3], b0, b1);
                mma_bf16(sc[j + 1], qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3], b2, b3);
            }
        }
        // scale + mask
        const int key0 = t * KT;
        const bool need_mask = key0 + KT > P;
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int h = e >> 1;
                float v = sc[j][e] * sl2;
                if (need_mask) {
                    const int key = key0 + j * 8 + t4 * 2 + (e & 1);
                    bool vis = key < P;
                    if (!vis && key < n_keys) {
                        const int b = key - P;
                        vis = p.anc ? ((anc_r[h][b >> 6] >> (b & 63)) & 1ull) : true;
                    }
                    if (!vis) v = -INFINITY;
                }
                sc[j][e] = v;
                mx[h] = fmaxf(mx[h], v);
            }
        }
        float corr[2], m_use[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
            const float m_new = fmaxf(m_r[h], mx[h]);
            m_use[h] = (m_new == -INFINITY) ? 0.f : m_new;
            corr[h] = exp2f(m_r[h] - m_use[h]);          // 0 when m_r was -inf
            m_r[h] = m_new;
        }
        float rs[2] = {0.f, 0.f};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float pv = exp2f(sc[j][e] - m_use[e >> 1]);
                sc[j][e] = pv;
                rs[e >> 1] += pv;
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) l_r[h] = l_r[h] * corr[h] + rs[h];
#pragma unroll
        for (int j = 0; j < DN; ++j) {
            o[j][0] *= corr[0]; o[j][1] *= corr[0];
            o[j][2] *= corr[1]; o[j][3] *= corr[1];
        }
        // O += P V : k-steps of 16 keys, n-tiles of 8 dims
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            const uint32_t a0 = pack_bf16(sc[2 * ks][0], sc[2 * ks][1]);
            const uint32_t a1 = pack_bf16(sc[2 * ks][2], sc[2 * ks][3]);
            const uint32_t a2 = pack_bf16(sc[2 * ks + 1][0], sc[2 * ks + 1][1]);
            const uint32_t a3 = pack_bf16(sc[2 * ks + 1][2], sc[2 * ks + 1][3]);
#pragma unroll
            for (int dn = 0; dn < DN; dn += 2) {
                uint32_t b0, b1, b2, b3;
                const int mtx = lane >> 3;
                ldsm_x4_t(smem_u32(cV + tile_off<D>(ks * 16 + (lane & 7) + (mtx & 1) * 8, dn + (mtx >> 1))), b0, b1, b2, b3);
                mma_bf16(o[dn], a0, a1, a2, a3, b0, b1);
                mma_bf16(o[dn + 1], a0, a1, a2, a3, b2, b3);
            }
        }
        __syncthreads();          // everyone done with this buffer before it is refilled
    }
    cp_async_wait<0>();

    // row sums across the 4 lanes that share a row
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        l_r[h] += __shfl_xor_sync(0xffffffffu, l_r[h], 1);
        l_r[h] += __shfl_xor_sync(0xffffffffu, l_r[h], 2);
    }

    if (p.S == 1) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int pr = qt * QT + warp * 16 + g8 + 8 * h;
            if (pr >= PR) continue;
            const int node = pr / G, g = pr % G;
            const float inv = 1.f / l_r[h];
            bf16 *dst = p.out + ((size_t)(s * p.T + node) * p.Hq + kvh * G + g) * D;
#pragma unroll
            for (int j = 0; j < DN; ++j)
                *reinterpret_cast<uint32_t *>(dst + j * 8 + t4 * 2) = pack_bf16(o[j][2 * h] * inv, o[j][2 * h + 1] * inv);
        }
        return;
    }

    // ---- partial results, then the last CTA of this (sequence, kv head, q tile) merges all splits
    const size_t row_base = ((size_t)s * p.Hkv + kvh) * PR;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int pr = qt * QT + warp * 16 + g8 + 8 * h;
        if (pr >= PR) continue;
        float *po = p.part_o + ((row_base + pr) * p.S + split) * D;
#pragma unroll
        for (int j = 0; j < DN; ++j)
            *reinterpret_cast<float2 *>(po + j * 8 + t4 * 2) = make_float2(o[j][2 * h], o[j][2 * h + 1]);
        if (t4 == 0) {
            float *pm = p.part_ml + ((row_base + pr) * p.S + split) * 2;
            pm[0] = m_r[h];
            pm[1] = l_r[h];
        }
    }
    __threadfence();
    __syncthreads();
    int32_t *ctr = p.counters + ((size_t)s * p.Hkv + kvh) * gridDim.x + qt;
    if (tid == 0) sh_last = (atomicAdd(ctr, 1) == p.S - 1);
    __syncthreads();
    if (!sh_last) return;
    __threadfence();
    const int rows = min(QT, PR - qt * QT);
    // weights w[r][sp] = 2^(m_sp - M) / sum_sp 2^(m_sp - M) l_sp, in a fixed split order
    for (int r = tid; r < rows; r += 128) {
        const float *pm = p.part_ml + ((row_base + qt * QT + r) * p.S) * 2;
        float M = -INFINITY;
        for (int sp = 0; sp < p.S; ++sp) M = fmaxf(M, __ldcg(pm + 2 * sp));
        float den = 0.f;
        for (int sp = 0; sp < p.S; ++sp) {
            const float w = exp2f(__ldcg(pm + 2 * sp) - M);
            sW[r * p.S + sp] = w;
            den += w * __ldcg(pm + 2 * sp + 1);
        }
        const float inv = 1.f / den;
        for (int sp = 0; sp < p.S; ++sp) sW[r * p.S + sp] *= inv;
    }
    __syncthreads();
    for (int it = tid; it < rows * (D / 2); it += 128) {
        const int r = it / (D / 2), c = (it % (D / 2)) * 2;
        const int pr = qt * QT + r;
        const float *po = p.part_o + ((row_base + pr) * p.S) * D + c;
        float a0 = 0.f, a1 = 0.f;
        for (int sp = 0; sp < p.S; ++sp) {
            const float2 v = __ldcg(reinterpret_cast<const float2 *>(po + (size_t)sp * D));
            const float w = sW[r * p.S + sp];
            a0 += w * v.x;
            a1 += w * v.y;
        }
        const int node = pr / G, g = pr % G;
        bf16 *dst = p.out + ((size_t)(s * p.T + node) * p.Hq + kvh * G + g) * D + c;
        *reinterpret_cast<uint32_t *>(dst) = pack_bf16(a0, a1);
    }
    if (tid == 0) *ctr = 0;
}

template <int D>
size_t attn_smem_bytes() { return (size_t)QT * D * 2 + 4 * (size_t)KT * D * 2 + (size_t)QT * 32 * sizeof(float); }

}  // namespace

int attention_q_tiles(int T, int G) { return (T * G + QT - 1) / QT; }

void launch_attention(const AttnParams &p, cudaStream_t st) {
    const int G = p.Hq / p.Hkv;
    dim3 grid(attention_q_tiles(p.T, G), p.Hkv, p.batch * p.S);
    if (p.d == 128) {
        static bool once = false;
        if (!once) {
            cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem_bytes<128>());
            once = true;
        }
        attn_kernel<128><<<grid, 128, attn_smem_bytes<128>(), st>>>(p);
    } else {
        static bool once = false;
        if (!once) {
            cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem_bytes<64>());
            once = true;
        }
        attn_kernel<64><<<grid, 128, attn_smem_bytes<64>(), st>>>(p);
    }
}

}  // namespace glance
