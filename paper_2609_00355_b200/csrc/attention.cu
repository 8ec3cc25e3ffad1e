// Split-KV paged attention of the packed tree rows (Definition 1: ancestor-masked target pass) and of
// the draft block (Section 3.2: every block slot sees the whole context and the whole block).
//
// One CTA = (64 packed query rows of one kv head, one key split), 16 warps.  The G query heads that
// share a kv head are packed into the row dimension (packed row = node * G + g), so each K/V page is
// fetched once per CTA for all of them.  Warp (rg, kg) owns query rows rg*16..+15 and, inside every
// 64-key tile (= one KV page), keys kg*16..+15: sixteen warps keep four warps per scheduler busy, which
// is what hides the latency of this short, dependent instruction stream.  Each warp runs its own
// online softmax (base 2, fp32) over its key subset; the four key groups are merged through shared
// memory at the end, and key splits are merged by the last CTA to arrive (no CTA waits on another).
// Keys 0..P-1 (committed context) are always visible; key P + j is visible to the row of node i iff
// bit j of anc[i] is set (or always, when no mask is given).
#include "kernels.cuh"

namespace glance {

namespace {

constexpr int QT = 64;          // packed query rows per CTA
constexpr int KT = kPage;       // keys per tile
constexpr int NTHREADS = 512;
constexpr int MAX_SPLITS = 16;
constexpr int PAGE_CACHE = 256;

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
struct Smem {
    static constexpr int Q_BYTES = QT * D * 2;
    static constexpr int KV_BYTES = KT * D * 2;                     // one K or V tile
    static constexpr int MERGE_FLOATS_PER_THREAD = D / 2 + 4;       // O fragment (D/8 n-tiles x 4) + m0,m1,l0,l1
    static constexpr int MERGE_BYTES = 3 * 4 * MERGE_FLOATS_PER_THREAD * 32 * 4;
    static constexpr int W_BYTES = QT * MAX_SPLITS * 4;
    // K/V ring of NBUF tiles each; the key-group merge area reuses the ring once the key loop is over
    static constexpr int NBUF = (D == 128) ? 5 : 8;
    static constexpr int RING_BYTES = 2 * NBUF * KV_BYTES;
    static constexpr int TOTAL = Q_BYTES + (RING_BYTES > MERGE_BYTES ? RING_BYTES : MERGE_BYTES) + W_BYTES;
};

template <int D>
__global__ void __launch_bounds__(NTHREADS, 1) attn_kernel(AttnParams p) {
    constexpr int CH = D / 8;                  // 16-byte chunks per row
    constexpr int KS = D / 16;                 // k-steps of QK^T
    constexpr int DN = D / 8;                  // n-tiles of the output
    constexpr int MF = Smem<D>::MERGE_FLOATS_PER_THREAD;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *sQ = smem;
    constexpr int NBUF = Smem<D>::NBUF;
    unsigned char *sK = sQ + Smem<D>::Q_BYTES;                         // NBUF buffers
    unsigned char *sV = sK + NBUF * Smem<D>::KV_BYTES;                 // NBUF buffers
    float *sM = reinterpret_cast<float *>(sK);                         // key-group merge area (aliases the ring)
    float *sW = reinterpret_cast<float *>(smem + Smem<D>::TOTAL - Smem<D>::W_BYTES);   // split-combine weights
    __shared__ int sh_pages[PAGE_CACHE];
    __shared__ int sh_last;

    // programmatic dependent launch: let the next kernel begin its prologue now; this kernel reads data of
    // its predecessors, so it waits for them before touching global memory
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int G = p.Hq / p.Hkv;
    const int PR = p.T * G;
    const int qt = blockIdx.x, kvh = blockIdx.y;
    const int s = blockIdx.z / p.S, split = blockIdx.z % p.S;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rg = warp & 3, kg = warp >> 2;
    const int g8 = lane >> 2, t4 = lane & 3;

    const int P = p.seq_len[s];
    const int n_keys = P + p.T;
    const int n_tiles = (n_keys + KT - 1) / KT;
    const int t_begin = (int)((long long)split * n_tiles / p.S);
    const int t_end = (int)((long long)(split + 1) * n_tiles / p.S);
    const int32_t *pt = p.page_table + (size_t)s * p.geom.max_pages_per_seq;

    // page ids of this split
    for (int i = tid; i < PAGE_CACHE && t_begin + i < t_end; i += NTHREADS) {
        const int t = t_begin + i;
        int page = (t < p.geom.max_pages_per_seq) ? pt[t] : -1;
        if (page < 0 || page >= p.geom.n_pages) {
            page = -1;
            set_status(p.status, GLANCE_E_BOUNDS);
        }
        sh_pages[i] = page;
    }
    // Q tile -> smem
    for (int it = tid; it < QT * CH; it += NTHREADS) {
        const int r = it / CH, c = it % CH;
        int pr = qt * QT + r;
        if (pr >= PR) pr = PR - 1;
        const int node = pr / G, g = pr % G;
        const bf16 *src = p.q + ((size_t)(s * p.T + node) * p.Hq + kvh * G + g) * D + c * 8;
        cp_async16(smem_u32(sQ + tile_off<D>(r, c)), src);
    }
    cp_async_commit();
    __syncthreads();                            // sh_pages visible

    auto load_tile = [&](int t, int buf) {
        int page;
        if (t - t_begin < PAGE_CACHE) page = sh_pages[t - t_begin];
        else {
            page = (t < p.geom.max_pages_per_seq) ? pt[t] : -1;
            if (page >= p.geom.n_pages) page = -1;
        }
        const bool ok = page >= 0;
        const bf16 *kbase = p.pool_layer + p.geom.row(ok ? page : 0, 0, kvh, 0);
        const bf16 *vbase = p.pool_layer + p.geom.row(ok ? page : 0, 1, kvh, 0);
        unsigned char *dK = sK + buf * Smem<D>::KV_BYTES, *dV = sV + buf * Smem<D>::KV_BYTES;
        const int valid = ok ? min(KT, n_keys - t * KT) : 0;
        for (int it = tid; it < KT * CH; it += NTHREADS) {
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
    };

    // prologue: NBUF-1 tiles in flight, one commit group per tile (empty groups keep the count uniform)
#pragma unroll
    for (int i = 0; i < NBUF - 1; ++i) {
        if (t_begin + i < t_end) load_tile(t_begin + i, i);
        cp_async_commit();
    }

    // the two rows (g8, g8+8) of this warp's 16 that this thread holds
    uint64_t anc0[2] = {0, 0}, anc1[2] = {0, 0};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        int pr = qt * QT + rg * 16 + g8 + 8 * h;
        if (pr >= PR) pr = PR - 1;
        if (p.anc) {
            const uint64_t *a = p.anc + ((size_t)s * p.T + pr / G) * p.W;
            anc0[h] = a[0];
            anc1[h] = p.W > 1 ? a[1] : 0ull;
        }
    }

    float o[DN][4];
#pragma unroll
    for (int j = 0; j < DN; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
    float m_r[2] = {-INFINITY, -INFINITY}, l_r[2] = {0.f, 0.f};
    const float sl2 = rsqrtf((float)D) * 1.4426950408889634f;

    for (int t = t_begin; t < t_end; ++t) {
        const int buf = (t - t_begin) % NBUF;
        cp_async_wait<NBUF - 2>();                       // tile t (and Q) have landed
        __syncthreads();                                 // ... for every thread; tile t-1's buffer is free
        if (t + NBUF - 1 < t_end) load_tile(t + NBUF - 1, (t - t_begin + NBUF - 1) % NBUF);
        cp_async_commit();
        const unsigned char *cK = sK + buf * Smem<D>::KV_BYTES, *cV = sV + buf * Smem<D>::KV_BYTES;

        // S = Q K^T for 16 rows x this warp's 16 keys
        float sc[2][4];
#pragma unroll
        for (int j = 0; j < 2; ++j) sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f;
        const int mtx = lane >> 3;
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) {
            uint32_t a0, a1, a2, a3, b0, b1, b2, b3;
            ldsm_x4(smem_u32(sQ + tile_off<D>(rg * 16 + (lane & 15), kk * 2 + (lane >> 4))), a0, a1, a2, a3);
            ldsm_x4(smem_u32(cK + tile_off<D>(kg * 16 + (lane & 7) + (mtx >> 1) * 8, kk * 2 + (mtx & 1))), b0, b1, b2, b3);
            mma_bf16(sc[0], a0, a1, a2, a3, b0, b1);
            mma_bf16(sc[1], a0, a1, a2, a3, b2, b3);
        }
        // scale + mask
        const int key0 = t * KT + kg * 16;
        const bool need_mask = t * KT + KT > P;
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < 2; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int h = e >> 1;
                float v = sc[j][e] * sl2;
                if (need_mask) {
                    const int key = key0 + j * 8 + t4 * 2 + (e & 1);
                    bool vis = key < P;
                    if (!vis && key < n_keys) {
                        const int b = key - P;
                        const uint64_t w = (b >> 6) ? anc1[h] : anc0[h];
                        vis = p.anc ? ((w >> (b & 63)) & 1ull) : true;
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
        for (int j = 0; j < 2; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float pv = exp2f(sc[j][e] - m_use[e >> 1]);
                sc[j][e] = pv;
                rs[e >> 1] += pv;
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) l_r[h] = l_r[h] * corr[h] + rs[h];
        if (corr[0] != 1.f || corr[1] != 1.f) {
#pragma unroll
            for (int j = 0; j < DN; ++j) {
                o[j][0] *= corr[0]; o[j][1] *= corr[0];
                o[j][2] *= corr[1]; o[j][3] *= corr[1];
            }
        }
        // O += P V : one k-step of 16 keys, n-tiles of 8 dims
        const uint32_t a0 = pack_bf16(sc[0][0], sc[0][1]);
        const uint32_t a1 = pack_bf16(sc[0][2], sc[0][3]);
        const uint32_t a2 = pack_bf16(sc[1][0], sc[1][1]);
        const uint32_t a3 = pack_bf16(sc[1][2], sc[1][3]);
#pragma unroll
        for (int dn = 0; dn < DN; dn += 2) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4_t(smem_u32(cV + tile_off<D>(kg * 16 + (lane & 7) + (mtx & 1) * 8, dn + (mtx >> 1))), b0, b1, b2, b3);
            mma_bf16(o[dn], a0, a1, a2, a3, b0, b1);
            mma_bf16(o[dn + 1], a0, a1, a2, a3, b2, b3);
        }
    }
    cp_async_wait<0>();
    __syncthreads();              // the ring is idle: its memory now serves the key-group merge

    // row sums across the 4 lanes that share a row
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        l_r[h] += __shfl_xor_sync(0xffffffffu, l_r[h], 1);
        l_r[h] += __shfl_xor_sync(0xffffffffu, l_r[h], 2);
    }

    // ---- merge the four key groups of each row group (fixed order kg = 0,1,2,3)
    if (kg > 0) {
        float *dst = sM + ((size_t)((kg - 1) * 4 + rg) * MF) * 32 + lane;
#pragma unroll
        for (int j = 0; j < DN; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) dst[(j * 4 + e) * 32] = o[j][e];
        }
        dst[(DN * 4 + 0) * 32] = m_r[0];
        dst[(DN * 4 + 1) * 32] = m_r[1];
        dst[(DN * 4 + 2) * 32] = l_r[0];
        dst[(DN * 4 + 3) * 32] = l_r[1];
    }
    __syncthreads();
    if (kg > 0) return;                       // warps 0..3 (one per row group) finish the job
    {
        float M[2] = {m_r[0], m_r[1]};
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            const float *src = sM + ((size_t)(k * 4 + rg) * MF) * 32 + lane;
            M[0] = fmaxf(M[0], src[(DN * 4 + 0) * 32]);
            M[1] = fmaxf(M[1], src[(DN * 4 + 1) * 32]);
        }
        float Mu[2] = {M[0] == -INFINITY ? 0.f : M[0], M[1] == -INFINITY ? 0.f : M[1]};
        float w0[2] = {exp2f(m_r[0] - Mu[0]), exp2f(m_r[1] - Mu[1])};
#pragma unroll
        for (int j = 0; j < DN; ++j) {
            o[j][0] *= w0[0]; o[j][1] *= w0[0];
            o[j][2] *= w0[1]; o[j][3] *= w0[1];
        }
        l_r[0] *= w0[0];
        l_r[1] *= w0[1];
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            const float *src = sM + ((size_t)(k * 4 + rg) * MF) * 32 + lane;
            const float wk[2] = {exp2f(src[(DN * 4 + 0) * 32] - Mu[0]), exp2f(src[(DN * 4 + 1) * 32] - Mu[1])};
#pragma unroll
            for (int j = 0; j < DN; ++j) {
#pragma unroll
                for (int e = 0; e < 4; ++e) o[j][e] += wk[e >> 1] * src[(j * 4 + e) * 32];
            }
            l_r[0] += wk[0] * src[(DN * 4 + 2) * 32];
            l_r[1] += wk[1] * src[(DN * 4 + 3) * 32];
        }
        m_r[0] = M[0];
        m_r[1] = M[1];
    }

    // from here on only warps 0..3 (128 threads) are alive; they synchronise on named barrier 1
    if (p.S == 1) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int pr = qt * QT + rg * 16 + g8 + 8 * h;
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
        const int pr = qt * QT + rg * 16 + g8 + 8 * h;
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
    asm volatile("bar.sync 1, 128;" ::: "memory");
    int32_t *ctr = p.counters + ((size_t)s * p.Hkv + kvh) * gridDim.x + qt;
    if (tid == 0) sh_last = (atomicAdd(ctr, 1) == p.S - 1);
    asm volatile("bar.sync 1, 128;" ::: "memory");
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
    asm volatile("bar.sync 1, 128;" ::: "memory");
    for (int it = tid; it < rows * (D / 4); it += 128) {
        const int r = it / (D / 4), c = (it % (D / 4)) * 4;
        const int pr = qt * QT + r;
        const float *po = p.part_o + ((row_base + pr) * p.S) * D + c;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sp = 0; sp < p.S; ++sp) {
            const float4 v = __ldcg(reinterpret_cast<const float4 *>(po + (size_t)sp * D));
            const float w = sW[r * p.S + sp];
            acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
        }
        const int node = pr / G, g = pr % G;
        bf16 *dst = p.out + ((size_t)(s * p.T + node) * p.Hq + kvh * G + g) * D + c;
        uint2 ov;
        ov.x = pack_bf16(acc.x, acc.y);
        ov.y = pack_bf16(acc.z, acc.w);
        *reinterpret_cast<uint2 *>(dst) = ov;
    }
    if (tid == 0) *ctr = 0;
}

void launch_pdl(void (*kernel)(AttnParams), dim3 grid, size_t smem, cudaStream_t st, const AttnParams &p) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(NTHREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, p);
}

}  // namespace

int attention_q_tiles(int T, int G) { return (T * G + QT - 1) / QT; }

int attention_splits(int T, int G, int Hkv, int batch) {
    const int ctas = attention_q_tiles(T, G) * Hkv * batch;
    int s = 148 / ctas;
    return s < 1 ? 1 : (s > MAX_SPLITS ? MAX_SPLITS : s);
}

void launch_attention(const AttnParams &p, cudaStream_t st) {
    const int G = p.Hq / p.Hkv;
    dim3 grid(attention_q_tiles(p.T, G), p.Hkv, p.batch * p.S);
    if (p.d == 128) {
        static bool once = false;
        if (!once) {
            cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<128>::TOTAL);
            once = true;
        }
        launch_pdl(attn_kernel<128>, grid, Smem<128>::TOTAL, st, p);
    } else {
        static bool once = false;
        if (!once) {
            cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<64>::TOTAL);
            once = true;
        }
        launch_pdl(attn_kernel<64>, grid, Smem<64>::TOTAL, st, p);
    }
}

}  // namespace glance
