// Split-KV paged attention on the 5th-generation tensor cores (tcgen05 + TMEM) for the packed tree rows
// (Definition 1: ancestor-masked target pass) and the draft block (Section 3.2).
//
// One CTA = (128 packed query rows of one kv head, one key split).  The G query heads that share a kv
// head are packed into the row dimension (packed row = node * G + g), so each K/V page is fetched once
// per CTA for all of them.  Per 64-key tile (= one KV page, TMA-loaded with 128-byte swizzle):
//     S[128 x 64]  = Q K^T          tcgen05.mma, A = Q (K-major, two bf16 terms hi + lo: the rounding of a query
//                                   would otherwise reach every score of its row), B = K page (K-major),
//                                   accumulator in TMEM
//     P            = 2^(S' - m)     softmax warps read S from TMEM (two threads per row), apply the scale and
//                                   the ancestor mask, write P back into TMEM over the scores as two bf16 terms
//                                   (hi in the first half of the tile's columns, lo in the second)
//     O[128 x d]  += P V            tcgen05.mma, A = P_hi, then P_lo, in tensor memory, B = V page (MN-major),
//                                   accumulator in TMEM
// The running reference maximum m of a row is only raised when a tile exceeds it by more than 2^8 (the
// accumulator is then rescaled in TMEM), so exponentials stay far inside fp32/bf16 range and O is almost
// never touched between tiles.  Warp roles: warp 0 = TMA producer, warp 1 = TMEM allocator + MMA issuer,
// warps 2..17 = softmax / epilogue.  The softmax warps form two groups: one takes the CTA's even key tiles, the
// other the odd ones, each with two S/P buffers, its own running maximum, row sums and accumulator in TMEM.  The
// scores of a group's next tile are issued a tile ahead into its other buffer, so a group goes from one tile
// straight to the next, and one group's exponentials run while the tensor pipe works for the other; the two
// accumulators are combined like two key splits when the loop ends.
// The key splits of a tile form a thread-block cluster and are merged through distributed shared memory
// (one asynchronous bulk copy per owner CTA, byte-counted on the owner's mbarrier).  Every mbarrier wait is
// bounded; a wait that gives up records GLANCE_E_TIMEOUT.
#include "kernels.cuh"
#include "tc_ptx.cuh"

namespace glance {

namespace {

using namespace tc;

constexpr int QT = 128;          // packed query rows per CTA (UMMA M)
constexpr int KT = kPage;        // keys per tile (UMMA N of S, K of P V)
constexpr int KS = 3;             // K page ring: scores are issued tiles ahead, so a K slot frees soon after its page lands
constexpr int VS = 2;             // V page ring: a V slot is held from the copy until the tile's second MMA
constexpr int MAX_SPLITS = 8;     // the splits of a tile form one thread-block cluster
constexpr float kRescaleThreshold = 8.f;   // log2 units

__device__ __forceinline__ float ex2_approx(float x) {   // 2^x, hardware approximation; 2^-inf = +0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
constexpr int P_TERMS = 2;       // bf16 terms of a probability (hi in the first half of the tile's S columns, lo in the second)
constexpr int NG = 2;            // softmax groups (tile i belongs to group i % NG; S, P and O buffers are per group)
constexpr int NCG = 2;           // column groups of a softmax group: threads per query row (a row's 64 scores are split over them)
constexpr int KPT = KT / NCG;    // keys per thread and tile
constexpr int GTHREADS = 128 * NCG;      // threads of one softmax group
constexpr int NSOFT = NG * GTHREADS;     // softmax / epilogue threads
constexpr int ECG = NSOFT / 128;         // column groups of the epilogue: a row's d outputs are split over them
constexpr int NTHREADS = 64 + NSOFT;
static_assert(NG == 2, "buffers are indexed by tile parity");
static_assert(KPT == 32, "the visibility bit set of a thread's keys is one 32-bit word");
static_assert(KPT % 32 == 0, "a thread writes its probabilities as 16-column chunks of bf16 pairs");

// 16 accumulator columns of a row, combined over the softmax groups: sum_g w[g] * O_g.  Warp-collective.  Only the
// first `groups` accumulators are read (a group without tiles never wrote its TMEM columns).
__device__ __forceinline__ void load_combined(uint32_t tmem_O, uint32_t addr, int d, int groups, const float (&w)[NG], float (&out)[16]) {
    uint32_t v[NG][16];
#pragma unroll
    for (int gi = 0; gi < NG; ++gi)
        if (gi < groups) tmem_ld16(tmem_O + (uint32_t)(gi * d) + addr, v[gi]);
    tmem_ld_wait();
#pragma unroll
    for (int j = 0; j < 16; ++j) out[j] = 0.f;
#pragma unroll
    for (int gi = 0; gi < NG; ++gi)
        if (gi < groups) {
#pragma unroll
            for (int j = 0; j < 16; ++j) out[j] = fmaf(w[gi], __uint_as_float(v[gi][j]), out[j]);
        }
}

template <int D>
struct Smem {
    static constexpr int SLABS = D / 64;                 // 64-element (128-byte) column slabs of a d-wide tile
    static constexpr int KV_BYTES = SLABS * KT * 128;    // one K or V page: 16 KB at d = 128
    static constexpr int Q_BYTES = 2 * SLABS * QT * 128; // both query planes: 64 KB at d = 128
    static constexpr int OPER_BYTES = Q_BYTES + (KS + VS) * KV_BYTES;   // Q, K ring, V ring (and merge staging)
    static constexpr int ROWF = D + 4;                   // floats per merged row: O, m, l, padding
    // split merge: rows received from the cluster's CTAs (each owner gets <= ceil(QT/S) rows from each of S CTAs)
    static constexpr int RECV_BYTES = (QT + MAX_SPLITS) * ROWF * 4;
    static constexpr int TOTAL = OPER_BYTES + RECV_BYTES + 1024;
    // tensor memory columns: two S buffers per group (4 x 64; P overwrites the first half of its S), one O (d) per group
    static constexpr uint32_t O_COL = 2 * NG * 64;
    static constexpr uint32_t TMEM_COLS = 512;
    static_assert(O_COL + NG * D <= TMEM_COLS, "tensor memory budget");
    static_assert(ROWF * 4 * QT <= OPER_BYTES, "merge staging fits the operand buffers");
};

struct alignas(8) AttnBars {
    uint64_t q_ready, k_full[KS], k_empty[KS], v_full[VS], v_empty[VS], s_full[2 * NG], p_full[2 * NG], o_done[NG], all_done, v_zero, merge;
    uint32_t tmem_base;
    int abort_flag;
};

template <int D>
__global__ void __launch_bounds__(NTHREADS, 1) attn_tc_kernel(const __grid_constant__ CUtensorMap map_kv, AttnParams p) {
    constexpr int SLABS = Smem<D>::SLABS;
    constexpr int CH = D / 8;                            // 16-byte chunks per row
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *sQ = smem;                                        // hi plane, lo plane
    unsigned char *sK = sQ + Smem<D>::Q_BYTES;                       // KS stages
    unsigned char *sV = sK + KS * Smem<D>::KV_BYTES;                 // VS stages
    __shared__ AttnBars bars;
    __shared__ float red[NG][2][NCG][QT];                 // per group: cross-column-group exchange of row maxima / sums
    __shared__ int quit[NG][2][4];                        // per group and lane quarter: leave the tile loop (decided by one thread)

    unsigned long long *trace = (p.trace && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) ? p.trace : nullptr;
    if (trace && threadIdx.x == 0) trace[0] = global_ns();
    if (p.trace && threadIdx.x == 0) atomicMin(p.trace + 14, (unsigned long long)global_ns());   // grid span: first start
    pdl_launch_dependents();
    const int G = p.Hq / p.Hkv;
    const int PR = p.T * G;
    const int qt = blockIdx.x, kvh = blockIdx.y;
    const int s = blockIdx.z / p.S, split = blockIdx.z % p.S;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        mbar_init(&bars.q_ready, NSOFT / 32);            // one arrival per softmax warp
        for (int b = 0; b < KS; ++b) {
            mbar_init(&bars.k_full[b], 1);
            mbar_init(&bars.k_empty[b], 1);
        }
        for (int b = 0; b < VS; ++b) {
            mbar_init(&bars.v_full[b], 1);
            mbar_init(&bars.v_empty[b], 1);
        }
        for (int b = 0; b < 2 * NG; ++b) {
            mbar_init(&bars.s_full[b], 1);
            mbar_init(&bars.p_full[b], GTHREADS / 32);   // one arrival per warp of the buffer's group
        }
        for (int b = 0; b < NG; ++b) mbar_init(&bars.o_done[b], 1);
        mbar_init(&bars.all_done, 1);
        mbar_init(&bars.v_zero, 1);
        mbar_init(&bars.merge, 1);
        bars.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (p.S > 1) {
            // split merge: this CTA owns a band of the tile's rows and receives that band from each of the S CTAs
            const int rpc = (QT + p.S - 1) / p.S;
            const int mine = max(0, min(rpc, QT - (int)cluster_rank() * rpc));
            if (mine > 0) mbar_expect_tx(&bars.merge, (uint32_t)(p.S * mine * Smem<D>::ROWF * 4));
        }
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars.tmem_base)), "r"(Smem<D>::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    if (p.S > 1) cluster_sync_all();                     // peers' merge barriers exist before anybody can signal them
    else __syncthreads();
    tc_fence_after();
    // S / P buffer of tile i: columns 64 (i & 3) (its parity is the group); O of group g: O_COL + d g
    const uint32_t tmem_S = bars.tmem_base, tmem_O = bars.tmem_base + Smem<D>::O_COL;
    volatile int *abort_flag = &bars.abort_flag;
    bool sm_ok = true;                                   // softmax warps: state carried into the split merge
    float sm_m = -INFINITY, sm_l = 0.f;
    float sm_w[NG] = {0.f, 0.f};                         // weights of the groups' accumulators in the combined row

    if (trace && threadIdx.x == 0) trace[1] = global_ns();
    // Sequence lengths and page tables only change in the commit kernel of the previous round, long finished:
    // they may be read before the dependency wait.  Pages entirely below seq_len - block_B hold committed
    // context that no kernel of this pass writes, so the producer prefetches them before the wait as well.
    const int P = p.seq_len[s];
    const int n_keys = P + p.T;
    const int n_tiles = (n_keys + KT - 1) / KT;
    // ceil-distribution: the extra tiles go to the first splits, because the last split already carries the
    // costlier masked tiles and the partial page
    const int t_begin = (int)(((long long)split * n_tiles + p.S - 1) / p.S);
    const int t_end = (int)(((long long)(split + 1) * n_tiles + p.S - 1) / p.S);
    const int nt = t_end - t_begin;
    const int32_t *pt = p.page_table + (size_t)s * p.geom.max_pages_per_seq;
    // second terms of queries / probabilities on pure-context tiles (see AttnParams::lo_skip)
    const bool skip_q_lo = (p.lo_skip & 1) && P >= p.lo_skip_min_keys;
    const bool skip_p_lo = (p.lo_skip & 2) && P >= p.lo_skip_min_keys;
    if (warp != 0) {
        pdl_wait();                                      // q, the tree rows' K/V and the outputs belong to other kernels
        if (trace && threadIdx.x == 64) trace[2] = global_ns();
    }

    if (warp == 0) {
        // ---------------- TMA producer: K pages and V pages in separate rings ----------------
        int issued_k = 0, issued_v = 0;
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_kv) : "memory");
            bool waited = false;
            // Rows written by this pass lie in [P - block_B, P + T): the head's refreshed context rows and the new
            // tree / block rows.  Pages entirely below that are committed context that no kernel of the pass writes,
            // so they may be fetched before the dependency wait.
            auto page_rows = [&](int i, int &krow, int &vrow) {
                const int t = t_begin + i;
                if (!waited && (t + 1) * KT > P - kMaxBlock) {
                    pdl_wait();
                    waited = true;
                }
                int page = (t < p.geom.max_pages_per_seq) ? pt[t] : -1;
                if (page < 0 || page >= p.geom.n_pages) {
                    page = 0;
                    set_status(p.status, GLANCE_E_BOUNDS);
                }
                krow = ((page * 2 + 0) * p.geom.n_kv_heads + kvh) * KT;
                vrow = ((page * 2 + 1) * p.geom.n_kv_heads + kvh) * KT;
            };
            // K and V pages advance independently, each as far ahead as its ring allows: one thread polls both rings
            uint64_t stall_t0 = 0;
            uint32_t spins = 0;
            while (issued_k < nt || issued_v < nt) {
                bool progressed = false;
                if (issued_k < nt && mbar_try_wait(&bars.k_empty[issued_k % KS], ((uint32_t)(issued_k / KS) & 1u) ^ 1u)) {
                    int krow, vrow;
                    page_rows(issued_k, krow, vrow);
                    const int slot = issued_k % KS;
                    mbar_expect_tx(&bars.k_full[slot], (uint32_t)Smem<D>::KV_BYTES);
#pragma unroll
                    for (int sl = 0; sl < SLABS; ++sl)
                        tma_load_2d(sK + slot * Smem<D>::KV_BYTES + sl * KT * 128, &map_kv, &bars.k_full[slot], sl * 64, krow);
                    ++issued_k;
                    progressed = true;
                }
                if (issued_v < nt && mbar_try_wait(&bars.v_empty[issued_v % VS], ((uint32_t)(issued_v / VS) & 1u) ^ 1u)) {
                    int krow, vrow;
                    page_rows(issued_v, krow, vrow);
                    const int slot = issued_v % VS;
                    mbar_expect_tx(&bars.v_full[slot], (uint32_t)Smem<D>::KV_BYTES);
#pragma unroll
                    for (int sl = 0; sl < SLABS; ++sl)
                        tma_load_2d(sV + slot * Smem<D>::KV_BYTES + sl * KT * 128, &map_kv, &bars.v_full[slot], sl * 64, vrow);
                    ++issued_v;
                    progressed = true;
                }
                if (progressed) {
                    stall_t0 = 0;
                } else if ((++spins & 63u) == 0) {
                    // bounded: no slot of either ring has come free for the whole limit, or another role gave up
                    if (*abort_flag) break;
                    const uint64_t now = global_ns();
                    if (stall_t0 == 0) stall_t0 = now;
                    else if (now - stall_t0 > kWaitLimitNs) {
                        *abort_flag = 1;
                        set_status(p.status, GLANCE_E_TIMEOUT);
                        break;
                    }
                }
            }
            if (!waited) pdl_wait();
        }
        // The page that holds the last key may continue with rows that belong to nobody (any bits, NaN included):
        // this warp zeroes them in the V slot once the page has landed, and tells the MMA issuer.  The wait is exact:
        // this thread issued the copy, and no later copy can follow into the slot before that tile's second MMA.
        const int last_valid = n_keys - (t_end - 1) * KT;       // keys of this CTA's last tile
        if (nt > 0 && last_valid < KT) {
            const int i = nt - 1, slot = i % VS;
            int got = 0;
            if (lane == 0) got = (issued_v == nt && mbar_wait(&bars.v_full[slot], (uint32_t)(i / VS) & 1u, abort_flag, p.status)) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (got) {
                unsigned char *v = sV + slot * Smem<D>::KV_BYTES;
                for (int it = lane; it < (KT - last_valid) * CH; it += 32) {
                    const int r = last_valid + it / CH, c = it % CH;
                    *reinterpret_cast<int4 *>(v + (c >> 3) * KT * 128 + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = make_int4(0, 0, 0, 0);
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars.v_zero);
            }
        }
        if (lane == 0) {
            if (*abort_flag) {
                // copies already issued must land before the CTA may exit
                for (int i = max(0, issued_k - KS); i < issued_k; ++i) {
                    const uint64_t t0 = global_ns();
                    while (!mbar_try_wait(&bars.k_full[i % KS], (uint32_t)(i / KS) & 1u))
                        if (global_ns() - t0 > kWaitLimitNs) break;
                }
                for (int i = max(0, issued_v - VS); i < issued_v; ++i) {
                    const uint64_t t0 = global_ns();
                    while (!mbar_try_wait(&bars.v_full[i % VS], (uint32_t)(i / VS) & 1u))
                        if (global_ns() - t0 > kWaitLimitNs) break;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // Tile i uses S / P buffer i & 3 (so a group alternates between its two buffers) and the accumulator of
        // group i & 1.  The scores of the first four tiles are issued up front; after P V of tile i the scores of
        // tile i + 4 follow into the buffer that P V has just read.
        if (lane == 0 && nt > 0) {
            const uint32_t idesc_s = umma_idesc(KT);              // M 128, N 64 keys
            const uint32_t idesc_o = umma_idesc_bmn(D);           // M 128, N d, B = V is MN-major
            const int planes = p.q_lo ? 2 : 1;
            auto issue_s = [&](int i) -> bool {
                const int b = i & 3, ks_slot = i % KS;    // S buffer in TMEM / K page slot in shared memory
                const int planes_i = (skip_q_lo && (t_begin + i + 1) * KT <= P) ? 1 : planes;
                if (!mbar_wait(&bars.k_full[ks_slot], (uint32_t)(i / KS) & 1u, abort_flag, p.status)) return false;
                tc_fence_after();
                const uint32_t kbase = smem_u32(sK + ks_slot * Smem<D>::KV_BYTES);
                for (int pl = 0; pl < planes_i; ++pl) {
                    const uint32_t qbase = smem_u32(sQ) + (uint32_t)(pl * SLABS * QT * 128);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const int sl = ks >> 2, kk = ks & 3;
                        umma_f16(tmem_S + (uint32_t)(b * 64), umma_desc(qbase + sl * QT * 128) + (uint64_t)(kk * 2),
                                 umma_desc(kbase + sl * KT * 128) + (uint64_t)(kk * 2), idesc_s, (pl | ks) > 0 ? 1u : 0u);
                    }
                }
                umma_commit(&bars.k_empty[ks_slot]);      // K page free once these MMAs have read it
                umma_commit(&bars.s_full[b]);
                return true;
            };
            bool ok = mbar_wait(&bars.q_ready, 0, abort_flag, p.status);
            for (int i = 0; i < 2 * NG && i < nt && ok; ++i) ok = issue_s(i);
            for (int i = 0; i < nt && ok; ++i) {
                const int b = i & 3, g = i & 1, vs = i % VS;
                if (!mbar_wait(&bars.p_full[b], (uint32_t)(i >> 2) & 1u, abort_flag, p.status)) { ok = false; break; }
                if (!mbar_wait(&bars.v_full[vs], (uint32_t)(i / VS) & 1u, abort_flag, p.status)) { ok = false; break; }
                // the rows after the last key have been zeroed by the producer warp
                if (i == nt - 1 && n_keys - (t_end - 1) * KT < KT && !mbar_wait(&bars.v_zero, 0, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t vbase = smem_u32(sV + vs * Smem<D>::KV_BYTES);
                const int p_terms = (skip_p_lo && (t_begin + i + 1) * KT <= P) ? 1 : P_TERMS;
                for (int pt = 0; pt < p_terms; ++pt)
#pragma unroll
                    for (int kk = 0; kk < KT / 16; ++kk)
                        umma_f16_ts(tmem_O + (uint32_t)(g * D), tmem_S + (uint32_t)(b * 64 + pt * (KT / 2) + kk * 8),
                                    umma_desc_mn(vbase + kk * 16 * 128, KT * 128), idesc_o, (i >= NG || pt > 0 || kk > 0) ? 1u : 0u);
                umma_commit(&bars.v_empty[vs]);           // V page free once these MMAs have read it
                umma_commit(&bars.o_done[g]);             // this group's O updated
                if (i + 2 * NG < nt && !issue_s(i + 2 * NG)) { ok = false; break; }
            }
            if (ok) umma_commit(&bars.all_done);         // every MMA of this CTA has completed when this barrier flips
        }
    } else {
        // ---------------- softmax / epilogue warps ----------------
        // 16 warps in two groups of 8.  Inside a group warp (q, cg) serves the TMEM lane quarter q (32 query rows)
        // and the column group cg: a row's 64 scores are split over NCG threads.  In the epilogue all 16 warps
        // split a row's d output columns four ways.
        const int q = warp & 3;                           // TMEM lane quarter this warp may access
        const int sw = warp - 2;                          // 0..15
        const int grp = sw / (4 * NCG);                   // softmax group: takes tiles i with i % NG == grp
        const int cg = (sw % (4 * NCG)) >> 2;             // column group inside the softmax group
        const int ecg = sw >> 2;                          // column group of the epilogue, 0..ECG-1
        const int row = q * 32 + lane;
        const int tsm = threadIdx.x - 64;                 // 0..NSOFT-1
        int pr = qt * QT + row;
        const bool row_valid = pr < PR;
        if (!row_valid) pr = PR - 1;
        const int node = pr / G, g = pr % G;
        // Q tile (both planes) -> shared memory in the K-major 128-byte-swizzled operand layout (async copies, all in
        // flight).  A thread keeps one 16-byte chunk column and walks rows NSOFT / CH apart: the row's source offset
        // (two integer divisions) is computed once per row and serves both planes.
        {
            static_assert(NSOFT % CH == 0 && QT % (NSOFT / CH) == 0, "a thread's chunks share one chunk column");
            constexpr int RSTEP = NSOFT / CH;             // rows between a thread's consecutive chunks
            const int c = tsm % CH;
            const uint32_t dst0 = smem_u32(sQ) + (uint32_t)((c >> 3) * QT * 128);
#pragma unroll
            for (int k = 0; k < QT / RSTEP; ++k) {
                const int r = tsm / CH + k * RSTEP;
                int prr = qt * QT + r;
                if (prr >= PR) prr = PR - 1;
                const size_t off = ((size_t)(s * p.T + prr / G) * p.Hq + kvh * G + prr % G) * D + c * 8;
                const uint32_t dst = dst0 + (uint32_t)(r * 128 + (((c & 7) ^ (r & 7)) << 4));
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(p.q + off));
                if (p.q_lo)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (uint32_t)(SLABS * QT * 128)), "l"(p.q_lo + off));
            }
        }
        asm volatile("cp.async.commit_group;" ::);
        // the row's ancestor words travel while the copies are in flight
        uint64_t anc0 = ~0ull, anc1 = ~0ull;               // no mask: every extra key is visible
        if (p.anc) {
            const uint64_t *a = p.anc + ((size_t)s * p.T + node) * p.W;
            anc0 = a[0];
            anc1 = p.W > 1 ? a[1] : 0ull;
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        fence_async_smem();
        __syncwarp();                                     // every lane's rows are written and fenced: one arrival per warp
        if (lane == 0) mbar_arrive(&bars.q_ready);
        if (trace && threadIdx.x == 64) trace[3] = global_ns();

        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        const float sl2 = rsqrtf((float)D) * 1.4426950408889634f;
        const uint32_t tmem_Og = tmem_O + (uint32_t)(grp * D);   // this group's accumulator
        const int st = grp;                               // V slot and accumulator barrier of every tile of this group
        float m_ref = -INFINITY, l_run = 0.f;             // l_run: this thread's share of the group's row sum
        bool ok = true;
        for (int i = grp; i < nt; i += NG) {
            const int t = t_begin + i;
            const int u = i >> 1;                         // this group's tile count so far
            const int sb = i & 3;                         // S / P buffer of the tile
            const uint32_t sph = (uint32_t)(i >> 2) & 1u; // phase of that buffer's barriers
            const int key0 = t * KT;
            ok = ok && mbar_wait(&bars.s_full[sb], sph, abort_flag, p.status);
            ok = __all_sync(0xffffffffu, ok);             // TMEM accesses are warp-collective
            if (trace && threadIdx.x == 64 && i == 0) trace[4] = global_ns();
            tc_fence_after();
            float sc[KPT];
            {
                uint32_t v[KPT / 16][16];
                if (ok) {
#pragma unroll
                    for (int c = 0; c < KPT / 16; ++c) tmem_ld16(tmem_S + lane_addr + (uint32_t)(sb * 64 + cg * KPT + c * 16), v[c]);
                    tmem_ld_wait();
                }
#pragma unroll
                for (int c = 0; c < KPT / 16; ++c)
#pragma unroll
                    for (int j = 0; j < 16; ++j) sc[c * 16 + j] = ok ? __uint_as_float(v[c][j]) : 0.f;
            }
            const bool need_mask = key0 + KT > P;
            const bool two_p = P_TERMS > 1 && !(skip_p_lo && !need_mask);   // this tile's probabilities keep their second term
            if (need_mask) {
                // visibility of this thread's KPT keys as one bit set: committed keys (< P) are visible, keys past
                // the last one are not, extra key b is visible if bit b of the row's ancestor set is (all of them
                // without a mask).  b0 = index of the first key among the extra keys; negative inside the context.
                const int b0 = key0 + cg * KPT - P;
                uint32_t vis;
                if (b0 >= 0) {
                    const uint64_t lo = b0 >= 64 ? anc1 : anc0, hi = b0 >= 64 ? 0ull : anc1;
                    const int sh = b0 & 63;
                    vis = (uint32_t)(sh == 0 ? lo : ((lo >> sh) | (hi << (64 - sh))));
                } else {
                    const int nctx = -b0;                 // leading committed keys
                    vis = nctx >= 32 ? 0xffffffffu : (((uint32_t)anc0 << nctx) | ((1u << nctx) - 1u));
                }
                const int n_valid = p.T - b0;             // keys of this thread that exist
                if (n_valid < 32) vis &= n_valid <= 0 ? 0u : ((1u << n_valid) - 1u);
#pragma unroll
                for (int j = 0; j < KPT; ++j) sc[j] = ((vis >> j) & 1u) ? sc[j] : -INFINITY;
            }
            // raw scores: the scale is folded into the exponent below
            float mt = fmaxf(sc[0], sc[1]);
#pragma unroll
            for (int j = 2; j < KPT; j += 2) mt = fmaxf(mt, fmaxf(sc[j], sc[j + 1]));
            // row maximum of the tile across the column groups (in scaled log2 units: sl2 > 0 keeps the order)
            mt *= sl2;
            red[grp][u & 1][cg][row] = mt;
            // Leaving the loop must be decided once per quarter: its warps meet at the barrier below every tile,
            // and the abort flag can change between two warps' reads.  One thread samples it before the barrier.
            if (cg == 0 && lane == 0) quit[grp][u & 1][q] = *abort_flag;
            asm volatile("bar.sync %0, %1;" ::"r"(2 + grp * 4 + q), "n"(32 * NCG) : "memory");   // only the group's warps of this lane quarter share rows
            if (quit[grp][u & 1][q]) break;               // a quarter that leaves stops arriving at p_full: every wait is bounded
            mt = red[grp][u & 1][0][row];
#pragma unroll
            for (int c = 1; c < NCG; ++c) mt = fmaxf(mt, red[grp][u & 1][c][row]);
            float factor = 1.f;
            if (m_ref == -INFINITY) {
                m_ref = mt;                               // nothing accumulated for this row yet
            } else if (mt > m_ref + kRescaleThreshold) {
                factor = exp2f(m_ref - mt);
                m_ref = mt;
            }
            if (__any_sync(0xffffffffu, factor != 1.f)) {
                if (i >= NG) {
                    // the accumulator may only be touched once the second MMA of the group's previous tile has landed.
                    // The parity wait is exact here: this tile's scores were issued behind the second MMA of the tile
                    // before that, so the barrier is at most one phase behind the awaited one and cannot be ahead of it.
                    ok = ok && mbar_wait(&bars.o_done[st], (uint32_t)(u - 1) & 1u, abort_flag, p.status);
                    ok = __all_sync(0xffffffffu, ok);
                }
                tc_fence_after();
                if (ok) {
                    l_run *= factor;
                    constexpr int RC = D / NCG;           // accumulator columns rescaled by this thread
#pragma unroll
                    for (int c = 0; c < RC; c += 16) {
                        uint32_t v[16];
                        tmem_ld16(tmem_Og + lane_addr + (uint32_t)(cg * RC + c), v);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * factor);
                        tmem_st16(tmem_Og + lane_addr + (uint32_t)(cg * RC + c), v);
                    }
                    tmem_st_wait();
                }
            }
            // P = 2^(S' - m_ref) as bf16 pairs, written over this tile's S columns (every thread of the row has its
            // scores in registers since the barrier above): hi terms in the first half, lo terms (what the hi term
            // lost to rounding) in the second; both are A operands of the second MMA
            float rs = 0.f;
            const float m_sub = (m_ref == -INFINITY) ? 0.f : m_ref;   // a fully masked row keeps -inf - 0 = -inf -> 2^-inf = 0
#pragma unroll
            for (int c = 0; c < KPT / 32; ++c) {
                uint32_t w[16], w2[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float a = sc[c * 32 + 2 * j], b = sc[c * 32 + 2 * j + 1];
                    const float pa = ex2_approx(fmaf(a, sl2, -m_sub));
                    const float pb = ex2_approx(fmaf(b, sl2, -m_sub));
                    rs += pa + pb;
                    __nv_bfloat162 h2 = __floats2bfloat162_rn(pa, pb);
                    w[j] = *reinterpret_cast<uint32_t *>(&h2);
                    if (two_p) {
                        __nv_bfloat162 l2 = __floats2bfloat162_rn(pa - __low2float(h2), pb - __high2float(h2));
                        w2[j] = *reinterpret_cast<uint32_t *>(&l2);
                    }
                }
                if (ok) {
                    tmem_st16(tmem_S + lane_addr + (uint32_t)(sb * 64 + cg * (KPT / 2) + c * 16), w);
                    if (two_p) tmem_st16(tmem_S + lane_addr + (uint32_t)(sb * 64 + KT / 2 + cg * (KPT / 2) + c * 16), w2);
                }
            }
            l_run += rs;
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();                                 // single arrivals of every thread would serialise on the barrier word
            if (lane == 0) mbar_arrive(&bars.p_full[sb]);  // always arrive: the MMA issuer counts one arrival per warp
            if (trace && threadIdx.x == 64 && i == 0) trace[5] = global_ns();
        }
        if (trace && threadIdx.x == 64) trace[6] = global_ns();
        // the groups' row sums and reference maxima meet here: every thread combines them in fixed order (this needs
        // no accumulator and runs while the last second MMA completes)
        asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
        red[grp][0][cg][row] = l_run;
        red[grp][1][cg][row] = m_ref;
        asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
        float gm[NG], gl[NG];
        float m_all = -INFINITY;
#pragma unroll
        for (int gi = 0; gi < NG; ++gi) {
            gm[gi] = red[gi][1][0][row];
            gl[gi] = red[gi][0][0][row];
#pragma unroll
            for (int c = 1; c < NCG; ++c) gl[gi] += red[gi][0][c][row];
            m_all = fmaxf(m_all, gm[gi]);
        }
        float l_row = 0.f;
#pragma unroll
        for (int gi = 0; gi < NG; ++gi) {
            // weight of the group's accumulator; a group without tiles, or with no visible key in this row, has none
            sm_w[gi] = (gi < nt && gm[gi] != -INFINITY) ? ex2_approx(gm[gi] - m_all) : 0.f;
            l_row += sm_w[gi] * gl[gi];
        }
        // The accumulators are read below by every softmax thread.  The per-group barrier cannot be used here: a
        // parity wait is only exact when the waiter is at most one phase behind, and a group does not observe every
        // phase of its accumulator barrier.  The issuer commits a one-shot barrier after its last MMA instead.
        if (ok && nt > 0) {
            ok = mbar_wait(&bars.all_done, 0, abort_flag, p.status);
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
        }
        ok = ok && (*abort_flag == 0);
        // ---------------- epilogue ----------------
        if (p.S == 1 && ok) {
            constexpr int OC = D / ECG;
            const float inv = 1.f / l_row;
            const size_t off = ((size_t)(s * p.T + node) * p.Hq + kvh * G + g) * D + ecg * OC;
#pragma unroll
            for (int c = 0; c < OC; c += 16) {
                float v[16];
                load_combined(tmem_O, lane_addr + (uint32_t)(ecg * OC + c), D, min(nt, NG), sm_w, v);
                if (row_valid) {
#pragma unroll
                    for (int j = 0; j < 16; j += 4)
                        store_two_term(p.out + off + c + j, p.out_lo ? p.out_lo + off + c + j : nullptr,
                                       make_float4(v[j] * inv, v[j + 1] * inv, v[j + 2] * inv, v[j + 3] * inv));
                }
            }
        }
        tc_fence_before();
        sm_ok = ok;
        sm_m = m_all;
        sm_l = l_row;
    }

    if (p.S > 1) {
        // ---------------- merge of the key splits inside the cluster (reduce-scatter by rows) ----------------
        // The S CTAs of one (sequence, kv head, q tile) form a cluster.  CTA `rank` owns rows [rank*RPC, +RPC).
        // Every CTA stages its unnormalised O rows with (m, l) in its own (now idle) operand buffers, then one
        // asynchronous shared-to-shared copy per owner ships that owner's band into the owner's receive region
        // and counts its bytes on the owner's merge barrier; the owner combines the S bands in split order.
        constexpr int ROWF = Smem<D>::ROWF;
        constexpr int OC = D / ECG;
        const int RPC = (QT + p.S - 1) / p.S;
        const uint32_t rank = cluster_rank();
        float *stage = reinterpret_cast<float *>(smem);
        unsigned char *recv = smem + Smem<D>::OPER_BYTES;
        if (trace && threadIdx.x == 64) trace[7] = global_ns();
        if (warp >= 2) {
            // this CTA's MMAs have all completed (o_done above) and every page it asked for has been consumed
            const int q = warp & 3, cg = (warp - 2) >> 2;   // epilogue column group
            const int row = q * 32 + lane;
            const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
            const bool live = nt > 0 && sm_ok;
            float *dst = stage + (size_t)row * ROWF + cg * OC;
#pragma unroll
            for (int c = 0; c < OC; c += 16) {
                float v[16];
                if (live) {
                    load_combined(tmem_O, lane_addr + (uint32_t)(cg * OC + c), D, min(nt, NG), sm_w, v);
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = 0.f;
                }
#pragma unroll
                for (int j = 0; j < 16; j += 4)
                    *reinterpret_cast<float4 *>(dst + c + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            }
            if (cg == 0) {
                stage[(size_t)row * ROWF + D] = live ? sm_m : -INFINITY;
                stage[(size_t)row * ROWF + D + 1] = live ? sm_l : 0.f;
            }
            fence_async_smem();                           // staged rows visible to the asynchronous copy engine
            asm volatile("bar.sync 1, %0;" ::"n"(NSOFT) : "memory");
            if (trace && threadIdx.x == 64) trace[8] = global_ns();
            if (warp == 2 && lane < p.S) {
                const uint32_t owner = (uint32_t)lane;
                const int rows = max(0, min(RPC, QT - (int)owner * RPC));
                if (rows > 0)
                    dsmem_bulk_copy(map_to_rank(smem_u32(recv) + (uint32_t)(rank * RPC * ROWF * 4), owner),
                                    smem_u32(stage) + (uint32_t)(owner * RPC * ROWF * 4), (uint32_t)(rows * ROWF * 4),
                                    map_to_rank(smem_u32(&bars.merge), owner));
            }
            if (trace && threadIdx.x == 64) trace[9] = global_ns();
            const int row_lo = (int)rank * RPC;
            const int own_rows = max(0, min(RPC, QT - row_lo));
            bool got = true;
            if (own_rows > 0) got = mbar_wait(&bars.merge, 0, abort_flag, p.status);
            // Everything bound for this CTA has landed: that is all its peers need to know before they may leave
            // (a CTA's staged rows are read by the copies it sent).  The matching wait is at the end of the kernel.
            cluster_arrive();
            if (trace && threadIdx.x == 64) trace[10] = global_ns();
            const int tsm = threadIdx.x - 64;
            const float *rows = reinterpret_cast<const float *>(recv);
            const int my_rows = got ? max(0, min(own_rows, PR - qt * QT - row_lo)) : 0;
            constexpr int SEG = D / 8;                    // items per row: two 4-float pieces, half a row apart
            for (int item = tsm; item < my_rows * SEG; item += NSOFT) {
                const int lr = item / SEG, c0 = (item % SEG) * 4, c1 = D / 2 + c0;
                const float *rp0 = rows + (size_t)lr * ROWF;
                const size_t sstride = (size_t)RPC * ROWF;      // floats between the same row of consecutive splits
                // all loads first (the values of up to MAX_SPLITS splits), then the arithmetic
                float ms[MAX_SPLITS], ls[MAX_SPLITS];
                float4 va[MAX_SPLITS], vb[MAX_SPLITS];
                float M = -INFINITY;
#pragma unroll
                for (int sp = 0; sp < MAX_SPLITS; ++sp) {
                    ms[sp] = -INFINITY; ls[sp] = 0.f;
                    va[sp] = vb[sp] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (sp < p.S) {
                        const float *rp = rp0 + sp * sstride;
                        ms[sp] = rp[D];
                        ls[sp] = rp[D + 1];
                        va[sp] = *reinterpret_cast<const float4 *>(rp + c0);
                        vb[sp] = *reinterpret_cast<const float4 *>(rp + c1);
                        M = fmaxf(M, ms[sp]);
                    }
                }
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), bcc = acc;
                float den = 0.f;
#pragma unroll
                for (int sp = 0; sp < MAX_SPLITS; ++sp) {  // split order: bit-reproducible
                    const float w = ex2_approx(ms[sp] - M);    // 2^-inf = 0 for an empty split
                    den += w * ls[sp];
                    acc.x += w * va[sp].x; acc.y += w * va[sp].y; acc.z += w * va[sp].z; acc.w += w * va[sp].w;
                    bcc.x += w * vb[sp].x; bcc.y += w * vb[sp].y; bcc.z += w * vb[sp].z; bcc.w += w * vb[sp].w;
                }
                const float inv = 1.f / den;
                const int prr = qt * QT + row_lo + lr;
                const size_t off = ((size_t)(s * p.T + prr / G) * p.Hq + kvh * G + prr % G) * D;
                store_two_term(p.out + off + c0, p.out_lo ? p.out_lo + off + c0 : nullptr,
                               make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv));
                store_two_term(p.out + off + c1, p.out_lo ? p.out_lo + off + c1 : nullptr,
                               make_float4(bcc.x * inv, bcc.y * inv, bcc.z * inv, bcc.w * inv));
            }
        } else {
            cluster_arrive();
        }
    }
    if (trace && threadIdx.x == 64) trace[11] = global_ns();
    if (p.trace && threadIdx.x == 64) atomicMax(p.trace + 15, (unsigned long long)global_ns());  // grid span: last end
    tc_fence_before();
    // no CTA leaves while its staged rows may still be read by a copy in flight, or a peer may still write to it
    if (p.S > 1) cluster_wait();
    else __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(bars.tmem_base), "r"(Smem<D>::TMEM_COLS) : "memory");
    }
}

template <int D>
cudaError_t launch_d(const AttnParams &p, const CUtensorMap &map_kv, dim3 grid, cudaStream_t st) {
    static bool once = false;
    if (!once) {
        cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::TOTAL);
        if (e != cudaSuccess) return e;
        once = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(NTHREADS, 1, 1);
    cfg.dynamicSmemBytes = Smem<D>::TOTAL;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;      // the key splits of one tile form a cluster
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = p.S;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, attn_tc_kernel<D>, map_kv, p);
}

// largest number of co-resident clusters of `cs` CTAs of this kernel (queried once per cluster size)
template <int D>
int max_active_clusters(int cs) {
    static int cache[MAX_SPLITS + 1] = {0};
    if (cache[cs] == 0) {
        cudaFuncSetAttribute(attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::TOTAL);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(1, 1, cs);
        cfg.blockDim = dim3(NTHREADS, 1, 1);
        cfg.dynamicSmemBytes = Smem<D>::TOTAL;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 1;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = cs;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, attn_tc_kernel<D>, &cfg) != cudaSuccess || n < 1) n = 148 / cs - 4;
        cache[cs] = n < 1 ? 1 : n;
    }
    return cache[cs];
}

}  // namespace

int attention_tc_q_tiles(int T, int G) { return (T * G + QT - 1) / QT; }

// Key splits per (sequence, kv head, q tile): the splits of a tile form a cluster, and all clusters of the
// launch should be resident at once (a second wave would double the kernel's latency).  A launch that cannot fit
// one wave split (several sequences) gets two splits: that halves the longest sequence's loop, which sets the
// launch's duration, while larger clusters lose more than they gain once clusters queue for SMs (a cluster starts
// only when enough SMs of one GPC are free together: 8 sequences of 1024-4096 positions took 100 / 84 / 102 / 154 us
// per layer with 1 / 2 / 4 / 8 splits).
int attention_tc_splits(int T, int G, int Hkv, int batch, int d) {
    const int base = attention_tc_q_tiles(T, G) * Hkv * batch;
    for (int s = MAX_SPLITS; s > 1; --s) {
        const int fit = d == 128 ? max_active_clusters<128>(s) : max_active_clusters<64>(s);
        if (base <= fit) return s;
    }
    return base <= 148 ? 2 : 1;
}

cudaError_t launch_attention_tc(const AttnParams &p, const CUtensorMap &map_kv, cudaStream_t st) {
    const int G = p.Hq / p.Hkv;
    dim3 grid(attention_tc_q_tiles(p.T, G), p.Hkv, p.batch * p.S);
    if (p.d == 128) return launch_d<128>(p, map_kv, grid, st);
    return launch_d<64>(p, map_kv, grid, st);
}

}  // namespace glance
