// Weight-streaming skinny GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), TMA-fed.
//
//   D[f][r] = sum_k W[f][k] * X[r][k]          ("swap-AB": weights are the UMMA M operand)
//
// One CTA owns a 128-row weight tile (UMMA M = 128) and up to 128 activation rows (UMMA N = NP, a
// multiple of 16) over one K range.  Weights are read from HBM exactly once; a ring of STAGES shared
// memory slots is filled by TMA (128-byte swizzle, one 64-wide k-slab per slot) and drained by
// tcgen05.mma issued from a single thread; the fp32 accumulator lives in TMEM and is read back by eight
// epilogue warps (one TMEM lane = one output feature, two warps per lane quarter).  Activations may be two-term
// (x = hi + lo, both bf16): the lo rows are NP more rows of the same B tile, and the epilogue adds the two
// accumulator halves.
//
// Warp roles: warp 0 = TMA producer, warp 1 = TMEM allocator + MMA issuer, warps 2..9 = epilogue.
// Epilogues: (0) fp32 split-K plane, (1) SwiGLU over 64 gate rows and their 64 up rows stacked into one tile,
// (2) row-wise arg-max over the vocabulary, merged across CTAs with a packed 64-bit atomic max,
// (3)/(4) split-K reduced inside a thread-block cluster through distributed shared memory, followed by
// residual add + norm statistics, or rotary embedding + paged K/V write.
// Every wait on an mbarrier is bounded; a wait that gives up records GLANCE_E_TIMEOUT, and the CTA
// drains and frees its TMEM before it returns.
#include <cuda.h>

#include "gemm_tc.cuh"
#include "tc_ptx.cuh"

namespace glance {

namespace {

using namespace tc;

constexpr int NEPI = 8;                  // epilogue warps: two per TMEM lane quarter, splitting the columns
constexpr int NTHR = 64 + 32 * NEPI;

struct alignas(8) Barriers {
    uint64_t full[12];
    uint64_t empty[12];
    uint64_t acc_ready;
    uint32_t tmem_base;
    int abort_flag;
};

// Philox4x32-10 (Salmon et al., SC 2011): the counter-based generator behind the sampling mode's noise field.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}
// standard Gumbel noise from one 32-bit word: u = ((w >> 9) + 0.5) 2^-23 lies strictly inside (0,1)
__device__ __forceinline__ float gumbel_from_word(uint32_t w) {
    const float u = ((float)(w >> 9) + 0.5f) * 1.1920928955078125e-07f;
    return -logf(-logf(u));
}

// MODE 0: fp32 planes              MODE 1: SwiGLU (64 gate + 64 up rows per tile)   MODE 2: arg-max (+ optional logits)
// MODE 3: split-K over a cluster, residual add + bf16 copy scaled by the next norm's gain + sum of squares
// MODE 4: split-K over a cluster, rotary embedding + q / paged K,V write
// MODE 5: per-row top-k candidates + log-sum-exp share of every 128-feature tile (draft LM head; + optional logits)
// Modes 0, 1, 2 and 4 multiply each activation row's results by 1/rms(row) when a.ssq is given: the rows
// they read are x * gain in bf16, and the row's sum of squares arrives as per-tile partial sums.
template <int MODE>
__global__ void __launch_bounds__(NTHR, (MODE == 0 || MODE == 2 || MODE == 5) ? 3 : 2) gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w,
                                                         const __grid_constant__ CUtensorMap map_x, TcGemmArgs a) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ Barriers bars;
    __shared__ float inv_rms[128];

    // MODE 1 stacks 64 gate rows and the matching 64 up rows into one 128-row weight tile (two TMA boxes)
    constexpr int FT = (MODE == 1) ? 64 : BM;            // output features per CTA
    constexpr bool CLUSTERED = (MODE == 3 || MODE == 4);
    const int NP = a.np;                                 // activation rows per CTA, padded to 16
    // With two-term activations (x = hi + lo, both bf16) the lo rows ride along as NP more rows of the B
    // operand: the accumulator gets NP more columns, which the epilogue adds to the first NP.
    const int NB = a.x_lo_row > 0 ? 2 * NP : NP;         // UMMA N
    const int stage_bytes = BM * 128 + NB * 128;
    const int stages = a.stages;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // grid = (weight tiles, K splits, 128-row blocks) -- or, with more than one row block, (row blocks, K splits,
    // weight tiles): CTAs are dispatched x-fastest, so the CTAs that stream the same weight tile for different row
    // blocks then start together and all but the first find the tile in L2 instead of reading HBM again
    const int tile_idx = a.rows_fastest ? blockIdx.z : blockIdx.x;
    const int f0 = tile_idx * FT;
    const int split = blockIdx.y;
    const int r0 = (a.rows_fastest ? blockIdx.x : blockIdx.z) * 128;
    const int ktiles = a.K / BK;
    const int kt0 = (int)((long long)split * ktiles / a.S), kt1 = (int)((long long)(split + 1) * ktiles / a.S);
    const int nk = kt1 - kt0;
    const uint32_t tmem_cols = a.tmem_cols;
    const uint64_t wait_limit = a.wait_limit_ns ? a.wait_limit_ns : kWaitLimitNs;

    // optional phase timestamps of CTA (0,0,0) (test hook; a.trace is nullptr in normal use)
    unsigned long long *trace = (a.trace && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) ? a.trace : nullptr;
    if (trace && threadIdx.x == 0) trace[0] = global_ns();
    if (a.trace && threadIdx.x == 0) atomicMin(a.trace + 14, (unsigned long long)global_ns());   // grid span: first start
    pdl_launch_dependents();
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
    if (trace && threadIdx.x == 0) trace[1] = global_ns();

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
            auto load_w = [&](int i, unsigned char *slot, uint64_t *bar) {
                const int k0 = (kt0 + i) * BK;
                if (MODE == 1) {
                    tma_load_2d(slot, &map_w, bar, k0, f0);                       // gate rows
                    tma_load_2d(slot + 64 * 128, &map_w, bar, k0, a.F + f0);     // up rows
                } else {
                    tma_load_2d(slot, &map_w, bar, k0, f0);
                }
            };
            // weights do not depend on earlier kernels: fill the ring with them before waiting on the predecessor
            const int pre = min(nk, stages);
            for (int i = 0; i < pre; ++i) {
                if (i + 1 == a.stall_kstep1) continue;        // test hook: this slot is never filled
                mbar_expect_tx(&bars.full[i], (uint32_t)stage_bytes);
                load_w(i, smem + (size_t)i * stage_bytes, &bars.full[i]);
            }
            pdl_wait();
            if (trace) trace[2] = global_ns();
            for (int i = 0; i < pre; ++i)
            {
                if (i + 1 == a.stall_kstep1) continue;
                unsigned char *xs = smem + (size_t)i * stage_bytes + BM * 128;
                tma_load_2d(xs, &map_x, &bars.full[i], (kt0 + i) * BK, r0);
                if (NB > NP) tma_load_2d(xs + NP * 128, &map_x, &bars.full[i], (kt0 + i) * BK, a.x_lo_row + r0);
            }
            int issued = pre;
            for (int i = pre; i < nk; ++i) {
                const int s = i % stages;
                const uint32_t ph = (uint32_t)(i / stages) & 1u;
                if (!mbar_wait(&bars.empty[s], ph ^ 1u, abort_flag, a.status, wait_limit)) break;
                if (i + 1 == a.stall_kstep1) continue;        // test hook (nothing issued: `issued` keeps its value)
                unsigned char *slot = smem + (size_t)s * stage_bytes;
                mbar_expect_tx(&bars.full[s], (uint32_t)stage_bytes);
                load_w(i, slot, &bars.full[s]);
                tma_load_2d(slot + BM * 128, &map_x, &bars.full[s], (kt0 + i) * BK, r0);
                if (NB > NP) tma_load_2d(slot + BM * 128 + NP * 128, &map_x, &bars.full[s], (kt0 + i) * BK, a.x_lo_row + r0);
                issued = i + 1;
            }
            if (*abort_flag) {
                // copies already issued must land before the CTA may exit
                for (int i = max(0, issued - stages); i < issued; ++i) {
                    if (i + 1 == a.stall_kstep1) continue;    // never issued
                    const uint64_t t0 = global_ns();
                    while (!mbar_try_wait(&bars.full[i % stages], (uint32_t)(i / stages) & 1u))
                        if (global_ns() - t0 > wait_limit) break;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc(NB);
            bool mok = true;
            for (int i = 0; i < nk && mok; ++i) {
                const int s = i % stages;
                const uint32_t ph = (uint32_t)(i / stages) & 1u;
                if (!mbar_wait(&bars.full[s], ph, abort_flag, a.status, wait_limit)) { mok = false; break; }
                if (trace && i == 0) trace[3] = global_ns();
                tc_fence_after();
                const uint32_t slot = smem_u32(smem + (size_t)s * stage_bytes);
                const uint64_t bdesc = umma_desc(slot + BM * 128);
                const uint64_t adesc = umma_desc(slot);
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)
                    umma_f16(tmem_base, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (i > 0 || k > 0) ? 1u : 0u);
                umma_commit(&bars.empty[s]);             // slot reusable once these MMAs have read it
            }
            if (mok) umma_commit(&bars.acc_ready);
        }
    } else {
        // ---------------- epilogue warps, part 1: row scales, then wait for the accumulator ----------------
        const int t = threadIdx.x - 64;                  // 0..255
        pdl_wait();                                      // everything below reads or writes data other kernels own
        if (MODE != 3) {
            float inv = 1.f;
            if (a.ssq && t < NP && r0 + t < a.R) {   // NP <= 128 < 256 epilogue threads
                float ss = 0.f;
                for (int i = 0; i < a.n_ssq; ++i) ss += __ldcg(a.ssq + (size_t)i * a.ssq_stride + r0 + t);
                inv = rsqrtf(ss / (float)a.K + a.eps);
            }
            if (t < 128) inv_rms[t] = inv;
        }
        if (nk > 0) ok = mbar_wait(&bars.acc_ready, 0, abort_flag, a.status, wait_limit);
        ok = __all_sync(0xffffffffu, ok);                // tcgen05.ld is warp-collective: decide as a warp
        tc_fence_after();
        asm volatile("bar.sync 1, 256;" ::: "memory");   // inv_rms visible to all epilogue warps
        if (trace && threadIdx.x == 64) trace[4] = global_ns();
        if (a.trace && threadIdx.x == 64 && nk > 0) {                                                 // main loop end: last / first CTA
            atomicMax(a.trace + 12, (unsigned long long)global_ns());
            atomicMin(a.trace + 13, (unsigned long long)global_ns());
        }
    }

    // ---------------- epilogue, part 2 ----------------
    // (a) every epilogue thread owns one TMEM lane (= one output feature of the tile) and moves its NP fp32
    //     results into a shared-memory tile laid out [row][feature] on top of the idle TMA ring -- its own
    //     ring, or, with split-K over a cluster, the ring of the CTA that owns the row;
    // (b) after a barrier the tile is processed one activation row per warp, four consecutive features per
    //     thread, so that every shared and global access is a 16-byte (fp32) or 8-byte (bf16) vector.
    const int q = warp & 3;                              // TMEM lane quarter an epilogue warp may read
    const int fl = q * 32 + lane;                        // feature within the tile (stage a)
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
    const uint32_t rank = CLUSTERED ? cluster_rank() : 0u;
    const int RP = CLUSTERED ? (NP + a.S - 1) / a.S : NP; // rows per owner CTA
    // Rows this CTA finishes (all NP, or its band of the cluster's reduce-scatter) and, for the first two rows
    // of each epilogue warp, the global operands of the row processing (residual, gain, rotary table, K/V row):
    // they are fetched here, ahead of the merge, so that their L2 latency hides under it.
    const int ew = warp - 2;                             // epilogue warp 0..7
    const int row_lo = (int)rank * RP;                   // first owned row (tile-local)
    const int my_rows = max(0, min(min(RP, NP - row_lo), a.R - r0 - row_lo));
    const int fo = 4 * lane;                             // first of this thread's four features (tile-local)
    float4 pre_a[2], pre_b[2], gain = make_float4(0.f, 0.f, 0.f, 0.f);
    long long pre_kv[2] = {-1, -1};
    pre_a[0] = pre_a[1] = pre_b[0] = pre_b[1] = gain;
    if (warp >= 2 && f0 + fo < a.Nout) {
        if (MODE == 3) {
            const uint2 gg = *reinterpret_cast<const uint2 *>(a.gain + f0 + fo);
            const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162 *>(&gg.x);
            const __nv_bfloat162 g23 = *reinterpret_cast<const __nv_bfloat162 *>(&gg.y);
            gain = make_float4(__low2float(g01), __high2float(g01), __low2float(g23), __high2float(g23));
#pragma unroll
            for (int u = 0; u < 2; ++u)
                if (ew + u * NEPI < my_rows)
                    pre_a[u] = __ldcg(reinterpret_cast<const float4 *>(a.x + (size_t)(r0 + row_lo + ew + u * NEPI) * a.Nout + f0 + fo));
        } else if (MODE == 4) {
            const int d = a.head_dim, half = d >> 1;
            const int h = (f0 + fo) / d, i = (f0 + fo) % d;
            const int ci = (i < half) ? i : i - half;
#pragma unroll
            for (int u = 0; u < 2; ++u)
                if (ew + u * NEPI < my_rows) {
                    const int rr = r0 + row_lo + ew + u * NEPI;
                    if (h < a.Hq + a.Hkv) {
                        pre_a[u] = *reinterpret_cast<const float4 *>(a.rope_cos + (size_t)rr * half + ci);
                        pre_b[u] = *reinterpret_cast<const float4 *>(a.rope_sin + (size_t)rr * half + ci);
                    }
                    if (h >= a.Hq) pre_kv[u] = a.kvrow[rr];
                }
        }
    }
    if (CLUSTERED) {
        cluster_sync_all();                              // every CTA's MMAs are done: all rings are idle
        if (trace && threadIdx.x == 64) trace[5] = global_ns();
    }
    if (warp >= 2) {
        // this CTA's plane inside an owner's ring, at the first of the lane quad's four features
        const uint32_t quad_base = smem_u32(smem) + (uint32_t)((rank * RP) * BM * 4) + (uint32_t)((q * 32 + (lane & ~3)) * 4);
        const int chalf = (warp - 2) >> 2;               // the two warps of a lane quarter alternate 16-column chunks
        for (int c = chalf * 16; c < NP; c += 32) {
            uint32_t v[16];
            if (nk > 0 && ok) {
                tmem_ld16(lane_addr + (uint32_t)c, v);
                if (NB > NP) {                           // hi part + lo part of the two-term activations
                    uint32_t w[16];
                    tmem_ld16(lane_addr + (uint32_t)(NP + c), w);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(w[j]));
                } else {
                    tmem_ld_wait();
                }
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = 0u;
            }
            if (CLUSTERED) {
                // 4 x 4 transposes inside each lane quad: lane i of a quad ends up with rows c+4m+i (m = 0..3) of
                // the quad's four consecutive features, so that a remote store carries 16 bytes instead of 4
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    uint32_t *e = v + 4 * m;
#pragma unroll
                    for (int k = 0; k < 4; k += 2) {
                        const uint32_t x = (lane & 1) ? e[k] : e[k + 1];
                        const uint32_t y = __shfl_xor_sync(0xffffffffu, x, 1);
                        if (lane & 1) e[k] = y; else e[k + 1] = y;
                    }
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        const uint32_t x = (lane & 2) ? e[k] : e[k + 2];
                        const uint32_t y = __shfl_xor_sync(0xffffffffu, x, 2);
                        if (lane & 2) e[k] = y; else e[k + 2] = y;
                    }
                    const int r = c + 4 * m + (lane & 3);
                    const uint32_t owner = (uint32_t)(r / RP);
                    const uint32_t dst = map_to_rank(quad_base + (uint32_t)((r - owner * RP) * BM * 4), owner);
                    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(e[0]), "r"(e[1]), "r"(e[2]), "r"(e[3]) : "memory");
                }
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) reinterpret_cast<float *>(smem)[(c + j) * BM + fl] = __uint_as_float(v[j]);
            }
        }
    }
    if (CLUSTERED) {
        if (trace && threadIdx.x == 64) trace[6] = global_ns();
        cluster_sync_all();                              // planes written and visible
        if (trace && threadIdx.x == 64) trace[7] = global_ns();
    } else if (warp >= 2) {
        asm volatile("bar.sync 1, 256;" ::: "memory");
    }
    if (warp >= 2 && ok) {
        const float *tile = reinterpret_cast<const float *>(smem);
        if (MODE == 0 || MODE == 2 || MODE == 5) {
            const bool vec = (a.ldy & 3) == 0;
            for (int r = ew; r < my_rows; r += NEPI) {
                const int rr = r0 + r;
                float4 v = *reinterpret_cast<const float4 *>(tile + r * BM + fo);
                const float sc = inv_rms[r];
                v.x *= sc; v.y *= sc; v.z *= sc; v.w *= sc;
                const int f = f0 + fo;
                if (MODE == 5) {
                    // Block slot 0 of every sequence is the root: its row is not a prediction (Section 3.2).
                    // Per row and tile: (max, sum of exponentials) for the log-sum-exp over the vocabulary, and the
                    // packed (value, id) keys that can still be among the row's k largest.  A key qualifies if it
                    // reaches a threshold that at least k entries of the row are known to reach.  The row keeps k
                    // running maxima in global memory, one per residue class of the tile index modulo k (every tile
                    // raises its class's maximum with atomicMax): the smallest of the k is such a threshold -- k
                    // entries of k different tiles reach it -- and with ~150 tiles per class it sits close to the
                    // row's true k-th largest value.  While a class is still empty, or if too many entries of this
                    // tile reach the bound, the tile falls back to its own bound, the k-th largest of its 32 lane
                    // maxima.  Which tiles emit what depends on timing; the merged result (the k largest keys,
                    // unique by id) does not.
                    if (rr % a.tk_B != 0) {
                        const bool in0 = f < a.Nout, in1 = f + 1 < a.Nout, in2 = f + 2 < a.Nout, in3 = f + 3 < a.Nout;
                        float m = -INFINITY;
                        if (in0) m = v.x;
                        if (in1) m = fmaxf(m, v.y);
                        if (in2) m = fmaxf(m, v.z);
                        if (in3) m = fmaxf(m, v.w);
                        const float lane_max = m;
                        m = warp_max(m);
                        float e = 0.f;
                        if (in0) e += __expf(v.x - m);
                        if (in1) e += __expf(v.y - m);
                        if (in2) e += __expf(v.z - m);
                        if (in3) e += __expf(v.w - m);
                        e = warp_sum(e);
                        const size_t slot = (size_t)tile_idx * a.R + rr;
                        if (lane == 0) {
                            a.tk_ml[2 * slot] = m;
                            a.tk_ml[2 * slot + 1] = e;
                        }
                        const uint32_t k0 = in0 ? float_key(v.x) : 0u, k1 = in1 ? float_key(v.y) : 0u;
                        const uint32_t k2 = in2 ? float_key(v.z) : 0u, k3 = in3 ? float_key(v.w) : 0u;
                        uint32_t T = lane < a.tk_k ? __ldcg(a.tk_thr + (size_t)rr * kTopkTileCap + lane) : 0xffffffffu;
                        T = __reduce_min_sync(0xffffffffu, T);
                        if (lane == 0 && m != -INFINITY) atomicMax(a.tk_thr + (size_t)rr * kTopkTileCap + tile_idx % a.tk_k, float_key(m));
                        auto count_at = [&](uint32_t t) {
                            return __popc(__ballot_sync(0xffffffffu, k0 >= t && in0)) + __popc(__ballot_sync(0xffffffffu, k1 >= t && in1)) +
                                   __popc(__ballot_sync(0xffffffffu, k2 >= t && in2)) + __popc(__ballot_sync(0xffffffffu, k3 >= t && in3));
                        };
                        int nhit = T ? count_at(T) : kTopkTileCap + 1;
                        if (nhit > kTopkTileCap) {
                            // the running bound is unset or loose: this tile's own bound, the k-th largest lane maximum
                            // (at least k entries of the tile reach it; k <= 16 <= 32 lanes)
                            uint32_t cur = lane_max == -INFINITY ? 0u : float_key(lane_max), tl = 0u;
                            for (int t = 0; t < a.tk_k; ++t) {
                                tl = __reduce_max_sync(0xffffffffu, cur);
                                const uint32_t holders = __ballot_sync(0xffffffffu, cur == tl);
                                if (lane == __ffs(holders) - 1) cur = 0u;
                            }
                            if (tl > T) T = tl;
                            nhit = T ? count_at(T) : kTopkTileCap + 1;
                        }
                        unsigned long long *out = a.tk_cand + slot * kTopkTileCap;
                        if (nhit <= kTopkTileCap) {
                            int at = 0;
                            const uint32_t below = (1u << lane) - 1u;
#define GLANCE_EMIT(kk, inb, val, id)                                                        \
                            {                                                                \
                                const bool hit = (inb) && (kk) >= T;                         \
                                const uint32_t hits = __ballot_sync(0xffffffffu, hit);       \
                                if (hit) out[at + __popc(hits & below)] = pack_val_id(val, id); \
                                at += __popc(hits);                                          \
                            }
                            GLANCE_EMIT(k0, in0, v.x, f) GLANCE_EMIT(k1, in1, v.y, f + 1) GLANCE_EMIT(k2, in2, v.z, f + 2) GLANCE_EMIT(k3, in3, v.w, f + 3)
#undef GLANCE_EMIT
                            if (lane == 0) a.tk_cnt[slot] = nhit;
                        } else {
                            // more than the slots hold (a tile full of equal values, or fewer than k entries): exact selection
                            const unsigned long long q0 = in0 ? pack_val_id(v.x, f) : 0ull, q1 = in1 ? pack_val_id(v.y, f + 1) : 0ull;
                            const unsigned long long q2 = in2 ? pack_val_id(v.z, f + 2) : 0ull, q3 = in3 ? pack_val_id(v.w, f + 3) : 0ull;
                            unsigned long long prev = ~0ull;
                            int n = 0;
                            for (int t = 0; t < a.tk_k; ++t) {
                                unsigned long long best = 0ull;
                                if (q0 < prev && q0 > best) best = q0;
                                if (q1 < prev && q1 > best) best = q1;
                                if (q2 < prev && q2 > best) best = q2;
                                if (q3 < prev && q3 > best) best = q3;
                                best = warp_max_u64(best);
                                if (best == 0ull) break;
                                if (lane == 0) out[t] = best;
                                prev = best;
                                ++n;
                            }
                            if (lane == 0) a.tk_cnt[slot] = n;
                        }
                    }
                }
                if (MODE == 0 || a.Y) {
                    float *dst = a.Y + (MODE == 0 ? (size_t)split * a.split_stride : 0) + (size_t)rr * a.ldy + f;
                    if (vec && f + 3 < a.Nout) *reinterpret_cast<float4 *>(dst) = v;
                    else {
                        if (f < a.Nout) dst[0] = v.x;
                        if (f + 1 < a.Nout) dst[1] = v.y;
                        if (f + 2 < a.Nout) dst[2] = v.z;
                        if (f + 3 < a.Nout) dst[3] = v.w;
                    }
                }
                if (MODE == 2) {
                    if (a.ent_out && rr % a.ent_N == 0) {
                        // root row of a sequence: this tile's share of the soft-max statistics behind the entropy
                        float m = -INFINITY;
                        if (f < a.Nout) m = v.x;
                        if (f + 1 < a.Nout) m = fmaxf(m, v.y);
                        if (f + 2 < a.Nout) m = fmaxf(m, v.z);
                        if (f + 3 < a.Nout) m = fmaxf(m, v.w);
                        m = warp_max(m);
                        float l = 0.f, t = 0.f, e;
                        if (f < a.Nout) { e = __expf(v.x - m); l += e; t += e * v.x; }
                        if (f + 1 < a.Nout) { e = __expf(v.y - m); l += e; t += e * v.y; }
                        if (f + 2 < a.Nout) { e = __expf(v.z - m); l += e; t += e * v.z; }
                        if (f + 3 < a.Nout) { e = __expf(v.w - m); l += e; t += e * v.w; }
                        l = warp_sum(l);
                        t = warp_sum(t);
                        if (lane == 0) {
                            float *dst = a.ent_part + ((size_t)tile_idx * a.ent_batch + rr / a.ent_N) * 3;
                            dst[0] = m; dst[1] = l; dst[2] = t;
                        }
                    }
                    if (a.sample_pos) {
                        // sampling mode: a draw from softmax(row * inv_temperature) is the arg-max of the row plus
                        // Gumbel noise; the noise of (token position, vocabulary id) is a fixed field, so the draw
                        // for a position does not depend on which row or round asks for it.  Ids f..f+3 are the
                        // four words of the block (f / 4, position of the predicted token).
                        const uint32_t pos = (uint32_t)(a.sample_pos[rr] + 1);
                        const uint4 w = philox4x32_10(make_uint4((uint32_t)(f >> 2), pos, 0u, 0u),
                                                      make_uint2((uint32_t)a.sample_seed, (uint32_t)(a.sample_seed >> 32)));
                        v.x = v.x * a.sample_inv_t + gumbel_from_word(w.x);
                        v.y = v.y * a.sample_inv_t + gumbel_from_word(w.y);
                        v.z = v.z * a.sample_inv_t + gumbel_from_word(w.z);
                        v.w = v.w * a.sample_inv_t + gumbel_from_word(w.w);
                    }
                    unsigned long long key = 0ull, k2;
                    if (f < a.Nout) key = pack_val_id(v.x, f);
                    if (f + 1 < a.Nout) { k2 = pack_val_id(v.y, f + 1); key = k2 > key ? k2 : key; }
                    if (f + 2 < a.Nout) { k2 = pack_val_id(v.z, f + 2); key = k2 > key ? k2 : key; }
                    if (f + 3 < a.Nout) { k2 = pack_val_id(v.w, f + 3); key = k2 > key ? k2 : key; }
                    key = warp_max_u64(key);
                    if (lane == 0) atomicMax(a.keys + rr, key);
                }
            }
        } else if (MODE == 1) {
            // tile features 0..63 are gate rows, 64..127 the matching up rows; item = (row, 4 gate features)
            const int t = threadIdx.x - 64;
            for (int item = t; item < my_rows * 16; item += 32 * NEPI) {
                const int r = item >> 4, fg = (item & 15) * 4;
                const float4 g = *reinterpret_cast<const float4 *>(tile + r * BM + fg);
                const float4 u = *reinterpret_cast<const float4 *>(tile + r * BM + 64 + fg);
                const float sc = inv_rms[r];
                const int f = f0 + fg;
                if (f < a.F) {          // F is a multiple of 4
                    const float g0 = g.x * sc, g1 = g.y * sc, g2 = g.z * sc, g3 = g.w * sc;
                    const float4 val = make_float4(g0 / (1.f + __expf(-g0)) * (u.x * sc), g1 / (1.f + __expf(-g1)) * (u.y * sc),
                                                   g2 / (1.f + __expf(-g2)) * (u.z * sc), g3 / (1.f + __expf(-g3)) * (u.w * sc));
                    store_two_term(a.act + (size_t)(r0 + r) * a.F + f, a.act_lo ? a.act_lo + (size_t)(r0 + r) * a.F + f : nullptr, val);
                }
            }
        } else if (MODE == 3) {
            const int f = f0 + fo;
            const bool valid = f < a.Nout;               // Nout is a multiple of 4
            int it = 0;
            for (int lr = ew; lr < my_rows; lr += NEPI, ++it) {
                const size_t o = (size_t)(r0 + row_lo + lr) * a.Nout + f;
                float4 xv = make_float4(0.f, 0.f, 0.f, 0.f);
                if (it == 0) xv = pre_a[0];
                else if (it == 1) xv = pre_a[1];
                else if (valid) xv = __ldcg(reinterpret_cast<const float4 *>(a.x + o));
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int k = 0; k < a.S; ++k) {          // split order: bit-reproducible
                    const float4 p = *reinterpret_cast<const float4 *>(tile + (size_t)(k * RP + lr) * BM + fo);
                    v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
                }
                float sq = 0.f;
                if (valid) {
                    xv.x += v.x; xv.y += v.y; xv.z += v.z; xv.w += v.w;
                    *reinterpret_cast<float4 *>(a.x + o) = xv;
                    store_two_term(a.xb + o, a.xb_lo ? a.xb_lo + o : nullptr,
                                   make_float4(xv.x * gain.x, xv.y * gain.y, xv.z * gain.z, xv.w * gain.w));
                    if (a.hidden_out) {
                        uint2 ob;
                        __nv_bfloat162 lo = __floats2bfloat162_rn(xv.x, xv.y);
                        __nv_bfloat162 hi = __floats2bfloat162_rn(xv.z, xv.w);
                        ob.x = *reinterpret_cast<uint32_t *>(&lo);
                        ob.y = *reinterpret_cast<uint32_t *>(&hi);
                        *reinterpret_cast<uint2 *>(a.hidden_out + o) = ob;
                    }
                    sq = ((xv.x * xv.x + xv.y * xv.y) + xv.z * xv.z) + xv.w * xv.w;
                }
                sq = warp_sum(sq);                       // one warp spans the tile's 128 features
                if (lane == 0) a.ssq_out[(size_t)tile_idx * a.ssq_stride + r0 + row_lo + lr] = sq;
            }
        } else {
            // MODE 4: q heads, then k heads, then v heads; rotary pairs (i, i + d/2) lie in the same tile
            const int d = a.head_dim, half = d >> 1;
            const int f = f0 + fo;
            const bool valid = f < a.Nout;
            const int h = f / d, i = f % d;              // the four features share head and half
            const bool is_q = h < a.Hq, is_k = !is_q && h < a.Hq + a.Hkv;
            const int pfo = (i < half) ? fo + half : fo - half;
            const int ci = (i < half) ? i : i - half;
            const int kvh = is_k ? h - a.Hq : h - a.Hq - a.Hkv;
            int it = 0;
            for (int lr = ew; lr < my_rows; lr += NEPI, ++it) {
                const int rr = r0 + row_lo + lr;
                float4 va = make_float4(0.f, 0.f, 0.f, 0.f), vb = va;
                for (int k = 0; k < a.S; ++k) {
                    const float *pl = tile + (size_t)(k * RP + lr) * BM;
                    const float4 pa = *reinterpret_cast<const float4 *>(pl + fo);
                    const float4 pb = *reinterpret_cast<const float4 *>(pl + pfo);
                    va.x += pa.x; va.y += pa.y; va.z += pa.z; va.w += pa.w;
                    vb.x += pb.x; vb.y += pb.y; vb.z += pb.z; vb.w += pb.w;
                }
                if (!valid) continue;
                const float sc = inv_rms[row_lo + lr];
                va.x *= sc; va.y *= sc; va.z *= sc; va.w *= sc;
                vb.x *= sc; vb.y *= sc; vb.z *= sc; vb.w *= sc;
                float4 out = va;
                if (is_q || is_k) {
                    const float4 cs = it == 0 ? pre_a[0] : it == 1 ? pre_a[1] : *reinterpret_cast<const float4 *>(a.rope_cos + (size_t)rr * half + ci);
                    const float4 sn = it == 0 ? pre_b[0] : it == 1 ? pre_b[1] : *reinterpret_cast<const float4 *>(a.rope_sin + (size_t)rr * half + ci);
                    if (i < half) {
                        out.x = va.x * cs.x - vb.x * sn.x; out.y = va.y * cs.y - vb.y * sn.y;
                        out.z = va.z * cs.z - vb.z * sn.z; out.w = va.w * cs.w - vb.w * sn.w;
                    } else {
                        out.x = va.x * cs.x + vb.x * sn.x; out.y = va.y * cs.y + vb.y * sn.y;
                        out.z = va.z * cs.z + vb.z * sn.z; out.w = va.w * cs.w + vb.w * sn.w;
                    }
                }
                if (is_q) {
                    // queries keep two bf16 terms: their rounding error would otherwise reach every score of the row
                    const size_t qo = ((size_t)rr * a.Hq + h) * d + i;
                    if (rr < a.Rq) store_two_term(a.q + qo, a.q_lo ? a.q_lo + qo : nullptr, out);
                } else {
                    __nv_bfloat162 lo = __floats2bfloat162_rn(out.x, out.y), hi = __floats2bfloat162_rn(out.z, out.w);
                    uint2 ob;
                    ob.x = *reinterpret_cast<uint32_t *>(&lo);
                    ob.y = *reinterpret_cast<uint32_t *>(&hi);
                    const long long base = it == 0 ? pre_kv[0] : it == 1 ? pre_kv[1] : a.kvrow[rr];
                    if (base >= 0)
                        *reinterpret_cast<uint2 *>(a.pool_layer + (size_t)base + (is_k ? 0 : a.v_off) + (size_t)kvh * a.head_stride + i) = ob;
                }
            }
        }
    }

    if (trace && threadIdx.x == 64) trace[8] = global_ns();
    if (a.trace && threadIdx.x == 64) {
        atomicMax(a.trace + 15, (unsigned long long)global_ns());                                 // grid span: last end
    }
    tc_fence_before();
    __syncthreads();
    if (trace && threadIdx.x == 0) trace[9] = global_ns();
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
            if (a.ent_out) {
                // entropy of every root row from the per-tile statistics: H = (M + log L) - T / L, merged in a fixed order
                __shared__ float red_m[NTHR / 32], red_l[NTHR / 32], red_t[NTHR / 32];
                const int tiles = (a.Nout + BM - 1) / BM;
                const int wid = threadIdx.x >> 5, ln = threadIdx.x & 31;
                for (int sq = 0; sq < a.ent_batch && sq * a.ent_N < a.R; ++sq) {
                    float M = -INFINITY, L = 0.f, T = 0.f;
                    for (int tl = threadIdx.x; tl < tiles; tl += blockDim.x) {
                        const float *src = a.ent_part + ((size_t)tl * a.ent_batch + sq) * 3;
                        const float m = __ldcg(src), l = __ldcg(src + 1), t = __ldcg(src + 2);
                        const float nm = fmaxf(M, m);
                        const float c0 = (M == -INFINITY) ? 0.f : __expf(M - nm), c1 = __expf(m - nm);
                        L = L * c0 + l * c1;
                        T = T * c0 + t * c1;
                        M = nm;
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const float m = __shfl_xor_sync(0xffffffffu, M, o), l = __shfl_xor_sync(0xffffffffu, L, o);
                        const float t = __shfl_xor_sync(0xffffffffu, T, o);
                        const float nm = fmaxf(M, m);
                        const float c0 = (M == -INFINITY) ? 0.f : __expf(M - nm), c1 = (m == -INFINITY) ? 0.f : __expf(m - nm);
                        L = L * c0 + l * c1;
                        T = T * c0 + t * c1;
                        M = nm;
                    }
                    if (ln == 0) { red_m[wid] = M; red_l[wid] = L; red_t[wid] = T; }
                    __syncthreads();
                    if (threadIdx.x == 0) {
                        float gm = -INFINITY;
                        for (int w = 0; w < NTHR / 32; ++w) gm = fmaxf(gm, red_m[w]);
                        float gl = 0.f, gt = 0.f;
                        for (int w = 0; w < NTHR / 32; ++w) {
                            const float c = (red_m[w] == -INFINITY) ? 0.f : __expf(red_m[w] - gm);
                            gl += red_l[w] * c;
                            gt += red_t[w] * c;
                        }
                        a.ent_out[sq] = (gm + logf(gl)) - gt / gl;
                    }
                    __syncthreads();
                }
            }
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
    cfg.blockDim = dim3(NTHR, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = (MODE == 3 || MODE == 4) ? grid.y : 1;     // the K splits of one tile form a cluster
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
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
    const int nb = a.x_lo_row > 0 ? 2 * a.np : a.np;
    const int stage_bytes = BM * 128 + nb * 128;
    // The ring stays under half of an SM's shared memory so that two CTAs fit per SM: a GPC then offers enough
    // CTA slots for every cluster of a launch to be resident in one wave, and one CTA's prologue and epilogue
    // overlap the other's streaming.
    const int tiles = mode == 1 ? (a.F + 63) / 64 : (a.Nout + BM - 1) / BM;
    // The LM heads have a few more tiles than two CTAs per SM take in four rounds (1188 against 1184 at the 7B
    // vocabulary): with a smaller ring three CTAs fit per SM and the last round is as full as the others.
    const bool three = (mode == 0 || mode == 2 || mode == 5) && tiles > 3 * 148;
    int stages = (int)(((three ? 72 : 100) * 1024) / stage_bytes);
    stages = stages > 12 ? 12 : (stages < 2 ? 2 : stages);
    a.stages = stages;
    uint32_t cols = 32;
    while ((int)cols < nb) cols <<= 1;
    a.tmem_cols = cols;
    const size_t smem = (size_t)stages * stage_bytes + 1024;
    const int row_blocks = (a.R + 127) / 128;
    a.rows_fastest = row_blocks > 1 ? 1 : 0;
    dim3 grid(a.rows_fastest ? row_blocks : tiles, a.S, a.rows_fastest ? tiles : row_blocks);
    if (mode == 3 || mode == 4) {
        // every CTA's ring must hold S planes of ceil(np/S) rows, and a cluster has at most 8 CTAs
        const size_t rp = (a.np + a.S - 1) / a.S;
        if (a.S > 8 || (size_t)a.S * rp * BM * 4 > (size_t)stages * stage_bytes) return cudaErrorInvalidValue;
    }
    if (mode == 0) return launch_mode<0>(a, map_w, map_x, smem, grid, st);
    if (mode == 1) return launch_mode<1>(a, map_w, map_x, smem, grid, st);
    if (mode == 2) return launch_mode<2>(a, map_w, map_x, smem, grid, st);
    if (mode == 3) return launch_mode<3>(a, map_w, map_x, smem, grid, st);
    if (mode == 5) return launch_mode<5>(a, map_w, map_x, smem, grid, st);
    return launch_mode<4>(a, map_w, map_x, smem, grid, st);
}

}  // namespace glance
