// Weight-streaming skinny GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), TMA-fed.
//
//   D[f][r] = sum_k W[f][k] * X[r][k]          ("swap-AB": weights are the UMMA M operand)
//
// One CTA owns a 128-row weight tile (UMMA M = 128) and up to 128 activation rows (UMMA N = NP, a
// multiple of 16) over one K range.  Weights are read from HBM exactly once; a ring of STAGES shared
// memory slots is filled by TMA (128-byte swizzle, one 64-wide k-slab per slot) and drained by
// tcgen05.mma issued from a single thread; the fp32 accumulator lives in TMEM and is read back by four
// epilogue warps (one TMEM lane = one output feature).
//
// Warp roles: warp 0 = TMA producer, warp 1 = TMEM allocator + MMA issuer, warps 2..5 = epilogue.
// Epilogues: (0) fp32 split-K plane, (1) SwiGLU over a gate tile and its up tile (two accumulators),
// (2) row-wise arg-max over the vocabulary, merged across CTAs with a packed 64-bit atomic max,
// (3)/(4) split-K reduced inside a thread-block cluster through distributed shared memory, followed by
// residual add + norm statistics, or rotary embedding + paged K/V write.
// Every wait on an mbarrier is bounded; a wait that gives up records GLANCE_E_TIMEOUT, and the CTA
// drains and frees its TMEM before it returns.
#include <cuda.h>

#include "gemm_tc.cuh"

namespace glance {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr uint64_t kWaitLimitNs = 1000ull * 1000ull * 1000ull;   // 1 s per wait

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the barrier did not flip within the limit or another role aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int32_t *status) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 63u) == 0) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                set_status(status, GLANCE_E_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}

// shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups 1024 B apart
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);        // start address
    d |= (uint64_t)1 << 16;                              // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                    // stride byte offset
    d |= (uint64_t)1 << 46;                              // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                              // SWIZZLE_128B
    return d;
}
// instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n
__host__ __device__ constexpr uint32_t umma_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

struct alignas(8) Barriers {
    uint64_t full[12];
    uint64_t empty[12];
    uint64_t acc_ready;
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of `local_addr` (a shared-memory address of this CTA) inside CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// MODE 0: fp32 planes              MODE 1: SwiGLU (two accumulators)      MODE 2: arg-max (+ optional logits)
// MODE 3: split-K over a cluster, residual add + bf16 copy scaled by the next norm's gain + sum of squares
// MODE 4: split-K over a cluster, rotary embedding + q / paged K,V write
// Modes 0, 1, 2 and 4 multiply each activation row's results by 1/rms(row) when a.ssq is given: the rows
// they read are x * gain in bf16, and the row's sum of squares arrives as per-tile partial sums.
template <int MODE>
__global__ void __launch_bounds__(192, (MODE >= 3) ? 2 : 1) gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w,
                                                         const __grid_constant__ CUtensorMap map_x, TcGemmArgs a) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ Barriers bars;
    __shared__ unsigned long long red_keys[4][128];
    __shared__ float inv_rms[128];
    __shared__ float red_sq[4][128];

    constexpr int NW = (MODE == 1) ? 2 : 1;              // weight tiles per stage
    constexpr bool CLUSTERED = (MODE >= 3);
    const int NP = a.np;                                 // UMMA N (activation rows, padded to 16)
    const int stage_bytes = NW * BM * 128 + NP * 128;
    const int stages = a.stages;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int f0 = blockIdx.x * BM;
    const int split = blockIdx.y;
    const int r0 = blockIdx.z * 128;
    const int ktiles = a.K / BK;
    const int kt0 = (int)((long long)split * ktiles / a.S), kt1 = (int)((long long)(split + 1) * ktiles / a.S);
    const int nk = kt1 - kt0;
    const uint32_t tmem_cols = a.tmem_cols;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&bars.full[s], 1);
            mbar_init(&bars.empty[s], 1);
        }
        mbar_init(&bars.acc_ready, 1);
        bars.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars.tmem_base)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars.tmem_base;
    volatile int *abort_flag = &bars.abort_flag;
    bool ok = true;                                      // epilogue warps: accumulator is valid

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
            int issued = 0;
            for (int i = 0; i < nk; ++i) {
                const int s = i % stages;
                const uint32_t ph = (uint32_t)(i / stages) & 1u;
                if (!mbar_wait(&bars.empty[s], ph ^ 1u, abort_flag, a.status)) break;
                unsigned char *slot = smem + (size_t)s * stage_bytes;
                mbar_expect_tx(&bars.full[s], (uint32_t)stage_bytes);
                const int k0 = (kt0 + i) * BK;
                tma_load_2d(slot, &map_w, &bars.full[s], k0, f0);
                if (NW == 2) tma_load_2d(slot + BM * 128, &map_w, &bars.full[s], k0, a.F + f0);
                tma_load_2d(slot + NW * BM * 128, &map_x, &bars.full[s], k0, r0);
                issued = i + 1;
            }
            if (*abort_flag) {
                // copies already issued must land before the CTA may exit
                for (int i = max(0, issued - stages); i < issued; ++i) {
                    const uint64_t t0 = global_ns();
                    while (!mbar_try_wait(&bars.full[i % stages], (uint32_t)(i / stages) & 1u))
                        if (global_ns() - t0 > kWaitLimitNs) break;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc(NP);
            bool mok = true;
            for (int i = 0; i < nk && mok; ++i) {
                const int s = i % stages;
                const uint32_t ph = (uint32_t)(i / stages) & 1u;
                if (!mbar_wait(&bars.full[s], ph, abort_flag, a.status)) { mok = false; break; }
                tc_fence_after();
                const uint32_t slot = smem_u32(smem + (size_t)s * stage_bytes);
                const uint64_t bdesc = umma_desc(slot + NW * BM * 128);
#pragma unroll
                for (int w = 0; w < NW; ++w) {
                    const uint64_t adesc = umma_desc(slot + w * BM * 128);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        umma_f16(tmem_base + (uint32_t)(w * NP), adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc,
                                 (i > 0 || k > 0) ? 1u : 0u);
                }
                umma_commit(&bars.empty[s]);             // slot reusable once these MMAs have read it
            }
            if (mok) umma_commit(&bars.acc_ready);
        }
    } else {
        // ---------------- epilogue warps, part 1: row scales, then wait for the accumulator ----------------
        const int t = threadIdx.x - 64;                  // 0..127
        if (MODE != 3) {
            float inv = 1.f;
            if (a.ssq && t < NP && r0 + t < a.R) {
                float ss = 0.f;
                for (int i = 0; i < a.n_ssq; ++i) ss += __ldcg(a.ssq + (size_t)i * a.ssq_stride + r0 + t);
                inv = rsqrtf(ss / (float)a.K + a.eps);
            }
            inv_rms[t] = inv;
        }
        if (MODE == 2) red_keys[warp & 3][lane] = red_keys[warp & 3][lane + 32] = red_keys[warp & 3][lane + 64] = red_keys[warp & 3][lane + 96] = 0ull;
        if (nk > 0) ok = mbar_wait(&bars.acc_ready, 0, abort_flag, a.status);
        ok = __all_sync(0xffffffffu, ok);                // tcgen05.ld is warp-collective: decide as a warp
        tc_fence_after();
        asm volatile("bar.sync 1, 128;" ::: "memory");   // inv_rms / red_keys visible to the four epilogue warps
    }

    const int q = warp & 3;                              // TMEM lane quarter an epilogue warp may read
    const int fl = q * 32 + lane;                        // feature within the tile
    const int f = f0 + fl;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);

    if (!CLUSTERED) {
        if (warp >= 2 && ok) {
            for (int c = 0; c < NP; c += 16) {
                uint32_t v[16];
                if (nk > 0) {
                    tmem_ld16(lane_addr + (uint32_t)c, v);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = 0u;
                }
                if (MODE == 0) {
                    float *Ys = a.Y + (size_t)split * a.split_stride;
                    if (f < a.Nout) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int r = r0 + c + j;
                            if (r < a.R) Ys[(size_t)r * a.ldy + f] = __uint_as_float(v[j]) * inv_rms[c + j];
                        }
                    }
                } else if (MODE == 1) {
                    uint32_t u[16];
                    tmem_ld16(lane_addr + (uint32_t)(NP + c), u);
                    tmem_ld_wait();
                    if (f < a.F) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int r = r0 + c + j;
                            const float g = __uint_as_float(v[j]) * inv_rms[c + j], up = __uint_as_float(u[j]) * inv_rms[c + j];
                            if (r < a.R) a.act[(size_t)r * a.F + f] = __float2bfloat16(g / (1.f + __expf(-g)) * up);
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int r = r0 + c + j;
                        const float val = __uint_as_float(v[j]) * inv_rms[c + j];
                        if (a.Y && f < a.Nout && r < a.R) a.Y[(size_t)r * a.ldy + f] = val;
                        unsigned long long key = (f < a.Nout) ? pack_val_id(val, f) : 0ull;
                        key = warp_max_u64(key);
                        if (lane == 0) red_keys[q][c + j] = key;
                    }
                }
            }
        }
        if (MODE == 2 && warp >= 2) {
            asm volatile("bar.sync 1, 128;" ::: "memory");
            const int t = threadIdx.x - 64;
            const int r = r0 + t;
            if (ok && t < NP && r < a.R) {
                unsigned long long k = red_keys[0][t];
                for (int w = 1; w < 4; ++w) k = red_keys[w][t] > k ? red_keys[w][t] : k;
                atomicMax(a.keys + r, k);
            }
        }
    } else {
        // ---------------- split-K over the cluster, reduce-scatter by rows: CTA `rank` owns activation rows
        // [rank*RP, rank*RP + RP) of the tile.  Every CTA ships, for each row, its fp32 partial results to the
        // owner's shared memory (planes [source split][row][feature], aliased onto the owner's idle TMA ring);
        // the owner adds the planes in split order and applies the fused epilogue to its rows ----------------
        const uint32_t rank = cluster_rank();
        const int RP = (NP + a.S - 1) / a.S;             // rows per owner
        cluster_sync_all();                              // every CTA's MMAs are done: all rings are idle
        if (warp >= 2) {
            const uint32_t local = smem_u32(smem) + (uint32_t)((rank * RP) * BM * 4) + (uint32_t)(fl * 4);
            for (int c = 0; c < NP; c += 16) {
                uint32_t v[16];
                if (nk > 0 && ok) {
                    tmem_ld16(lane_addr + (uint32_t)c, v);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = 0u;
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int r = c + j;
                    const uint32_t owner = (uint32_t)(r / RP);
                    st_cluster_f32(map_to_rank(local + (uint32_t)((r - owner * RP) * BM * 4), owner), __uint_as_float(v[j]));
                }
            }
        }
        cluster_sync_all();                              // planes written and visible
        if (warp >= 2) {
            const float *planes = reinterpret_cast<const float *>(smem);
            const int row_lo = (int)rank * RP;                                   // first owned row (tile-local)
            const int my_rows = max(0, min(min(RP, NP - row_lo), a.R - r0 - row_lo));
            if (MODE == 3) {
                const bool valid = f < a.Nout;
                const float gain = valid ? __bfloat162float(a.gain[f]) : 0.f;
                for (int rb = 0; rb < my_rows; rb += 8) {
                    float xv[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        xv[j] = (valid && rb + j < my_rows) ? __ldcg(a.x + (size_t)(r0 + row_lo + rb + j) * a.Nout + f) : 0.f;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int lr = rb + j;
                        if (lr >= my_rows) break;            // uniform across the warp
                        float v = 0.f;
                        for (int k = 0; k < a.S; ++k) v += planes[(size_t)(k * RP + lr) * BM + fl];
                        float sq = 0.f;
                        if (valid) {
                            const size_t o = (size_t)(r0 + row_lo + lr) * a.Nout + f;
                            const float xn = xv[j] + v;
                            a.x[o] = xn;
                            a.xb[o] = __float2bfloat16(xn * gain);
                            if (a.hidden_out) a.hidden_out[o] = __float2bfloat16(xn);
                            sq = xn * xn;
                        }
                        sq = warp_sum(sq);
                        if (lane == 0) red_sq[q][lr] = sq;
                    }
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const int t = threadIdx.x - 64;
                if (t < my_rows)
                    a.ssq_out[(size_t)blockIdx.x * a.ssq_stride + r0 + row_lo + t] =
                        ((red_sq[0][t] + red_sq[1][t]) + red_sq[2][t]) + red_sq[3][t];
            } else {
                const int d = a.head_dim, half = d >> 1;
                const int h = f / d, i = f % d;
                const bool is_q = h < a.Hq, is_k = !is_q && h < a.Hq + a.Hkv, valid = f < a.Nout;
                const int pfl = (i < half) ? fl + half : fl - half;          // rotary partner, same tile
                const int ci = (i < half) ? i : i - half;
                const int kvh = is_k ? h - a.Hq : h - a.Hq - a.Hkv;
                for (int rb = 0; rb < my_rows; rb += 8) {
                    float cs[8], sn[8];
                    long long base[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int rr = r0 + row_lo + rb + j;
                        const bool live = valid && rb + j < my_rows;
                        cs[j] = (live && !(!is_q && !is_k)) ? a.rope_cos[(size_t)rr * half + ci] : 1.f;
                        sn[j] = (live && !(!is_q && !is_k)) ? a.rope_sin[(size_t)rr * half + ci] : 0.f;
                        base[j] = (live && !is_q) ? a.kvrow[rr] : -1;
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int lr = rb + j;
                        if (lr >= my_rows) break;
                        const int rr = r0 + row_lo + lr;
                        float va = 0.f, vb = 0.f;
                        for (int k = 0; k < a.S; ++k) {
                            const float *pl = planes + (size_t)(k * RP + lr) * BM;
                            va += pl[fl];
                            vb += pl[pfl];
                        }
                        if (!valid) continue;
                        va *= inv_rms[row_lo + lr];
                        vb *= inv_rms[row_lo + lr];
                        const float out = (is_q || is_k) ? ((i < half) ? va * cs[j] - vb * sn[j] : va * cs[j] + vb * sn[j]) : va;
                        if (is_q) {
                            if (rr < a.Rq) a.q[((size_t)rr * a.Hq + h) * d + i] = __float2bfloat16(out);
                        } else if (base[j] >= 0) {
                            a.pool_layer[(size_t)base[j] + (is_k ? 0 : a.v_off) + (size_t)kvh * a.head_stride + i] = __float2bfloat16(out);
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
    if (MODE == 2) {
        // the last CTA to finish turns the merged keys into token ids and re-arms keys and counter
        __shared__ int is_last;
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) is_last = (atomicAdd(a.counter, 1) == (int)(gridDim.x * gridDim.y * gridDim.z) - 1);
        __syncthreads();
        if (is_last) {
            __threadfence();
            for (int r = threadIdx.x; r < a.R; r += blockDim.x) {
                const unsigned long long k = __ldcg(a.keys + r);
                a.argmax[r] = unpack_id(k);
                a.keys[r] = 0ull;
            }
            if (threadIdx.x == 0) *a.counter = 0;
        }
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

template <int MODE>
cudaError_t launch_mode(const TcGemmArgs &a, const CUtensorMap &mw, const CUtensorMap &mx, size_t smem, dim3 grid,
                        cudaStream_t st) {
    static bool once = false;
    if (!once) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        if (e != cudaSuccess) return e;
        once = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(192, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = (MODE >= 3) ? grid.y : 1;     // the K splits of one tile form a cluster
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<MODE>, mw, mx, a);
}

}  // namespace

bool tc_make_map(CUtensorMap *map, const void *base, uint64_t inner, uint64_t rows, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    if (((uintptr_t)base & 15) != 0 || (inner * 2) % 16 != 0) return false;
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {inner * 2};
    cuuint32_t box[2] = {BK, box_rows};
    cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int tc_row_pad(int R) {
    const int r = R > 128 ? 128 : R;
    return (r + 15) / 16 * 16;
}

cudaError_t launch_gemm_tc(int mode, TcGemmArgs a, const CUtensorMap &map_w, const CUtensorMap &map_x, cudaStream_t st) {
    a.np = tc_row_pad(a.R);
    const int nw = (mode == 1) ? 2 : 1;
    const int stage_bytes = nw * BM * 128 + a.np * 128;
    // Clustered modes keep the ring under half of an SM's shared memory so that two CTAs fit per SM: a GPC
    // then offers enough CTA slots for every cluster of the launch to be resident in one wave.
    int stages = (int)(((mode >= 3 ? 100 : 212) * 1024) / stage_bytes);
    stages = stages > 12 ? 12 : (stages < 2 ? 2 : stages);
    a.stages = stages;
    uint32_t cols = 32;
    while ((int)cols < nw * a.np) cols <<= 1;
    a.tmem_cols = cols;
    const size_t smem = (size_t)stages * stage_bytes + 1024;
    const int tiles = ((mode == 1 ? a.F : a.Nout) + BM - 1) / BM;
    dim3 grid(tiles, a.S, (a.R + 127) / 128);
    if (mode >= 3) {
        // every CTA's ring must hold S planes of ceil(np/S) rows, and a cluster has at most 8 CTAs
        const size_t rp = (a.np + a.S - 1) / a.S;
        if (a.S > 8 || (size_t)a.S * rp * BM * 4 > (size_t)stages * stage_bytes) return cudaErrorInvalidValue;
    }
    if (mode == 0) return launch_mode<0>(a, map_w, map_x, smem, grid, st);
    if (mode == 1) return launch_mode<1>(a, map_w, map_x, smem, grid, st);
    if (mode == 2) return launch_mode<2>(a, map_w, map_x, smem, grid, st);
    if (mode == 3) return launch_mode<3>(a, map_w, map_x, smem, grid, st);
    return launch_mode<4>(a, map_w, map_x, smem, grid, st);
}

}  // namespace glance
