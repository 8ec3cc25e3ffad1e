// Candidate-tree construction (Algorithm 1 lines 2-3) and greedy walk + KV commit (lines 5-12).
#include "kernels.cuh"

namespace glance {

// ------------------------------------------------------------------------------------------
// Best-first tree builder: one warp per sequence.
//
// Keeps the min(N-1, sum_l k^l) prefixes of highest score under the total order
// (score desc, depth asc, path key asc).  The frontier holds, for every kept node, its rank-0 child and
// its next-rank sibling; both score no higher than the node (log-probabilities are <= 0 and
// non-increasing in rank, fp32 addition is monotone), so repeatedly popping the best frontier entry
// enumerates the order exactly.  A node's score is one fp32 add from its parent's score.
// ------------------------------------------------------------------------------------------
struct Cand {
    float score;
    int depth;
    unsigned long long key;
};
__device__ __forceinline__ bool cand_before(const Cand &a, const Cand &b) {
    if (a.score != b.score) return a.score > b.score;
    if (a.depth != b.depth) return a.depth < b.depth;
    return a.key < b.key;
}

// The frontier lives in registers, entry e in slot e / 32 of lane e % 32; every lane follows the whole loop
// redundantly (counts, the popped entry, the two new entries), so that a pop needs one hardware warp max over the
// 32-bit score images, a handful of shuffles and no barrier: the only shared-memory traffic is the candidate
// tables (read-only) and the node arrays (each written and later re-read by the same lane).
// A pop replaces the entry by its child in place and appends its next sibling, so the frontier never exceeds N
// entries and nothing is moved.
// An entry is (sk, t, meta, ps): sk = order-preserving image of the score, t = tie word ((15 - depth) << 60 |
// complemented 60-bit path key), meta = depth | rank << 4 | parent << 8, ps = the parent's score (a next-rank
// sibling's score is one fp32 add from it).  Larger (sk, t) is popped first.
constexpr int kFrSlots = (kMaxTreeN + 4 + 31) / 32;      // 5 slots cover a frontier of N + 1 <= 129 entries

__global__ void __launch_bounds__(32) build_tree_kernel(int N, int L, int k, const int32_t *root, const int32_t *ids,
                                                        const float *lp, glance_tree out) {
    __shared__ float n_score[kMaxTreeN];
    __shared__ int n_token[kMaxTreeN], n_parent[kMaxTreeN], n_depth[kMaxTreeN], n_rank[kMaxTreeN];
    __shared__ unsigned long long n_anc[kMaxTreeN * 2];
    __shared__ float s_lp[kMaxBlock * kMaxTopk];
    __shared__ int s_id[kMaxBlock * kMaxTopk];
    const int s = blockIdx.x, lane = threadIdx.x;
    const int W = (N + 63) >> 6;
    const int32_t *sid = ids + (size_t)s * L * k;
    const float *slp = lp + (size_t)s * L * k;
    for (int e = lane; e < L * k; e += 32) {
        s_lp[e] = slp[e];
        s_id[e] = sid[e];
    }
    const int32_t root_tok = root[s];
    __syncwarp();

    // five slots as named scalars (arrays, even with unrolled compile-time indices, ended up in local memory)
    static_assert(kFrSlots == 5, "the slot macros below spell out five slots");
    uint32_t sk0 = 0u, sk1 = 0u, sk2 = 0u, sk3 = 0u, sk4 = 0u, me0 = 0u, me1 = 0u, me2 = 0u, me3 = 0u, me4 = 0u;
    unsigned long long tw0 = 0ull, tw1 = 0ull, tw2 = 0ull, tw3 = 0ull, tw4 = 0ull;
    float ps0 = 0.f, ps1 = 0.f, ps2 = 0.f, ps3 = 0.f, ps4 = 0.f;
    const bool deep = N > 94;                            // the frontier (<= N + 1 entries) reaches slots 3 and 4
#define GLANCE_SLOTS(OP) OP(0, sk0, tw0, me0, ps0) OP(1, sk1, tw1, me1, ps1) OP(2, sk2, tw2, me2, ps2) \
    if (deep) { OP(3, sk3, tw3, me3, ps3) OP(4, sk4, tw4, me4, ps4) }
#define GLANCE_PUT_OP(u, sk, tw, me, ps) if (pmine && pslot == u) { sk = psk; tw = ptw; me = pmeta; ps = pps; }
#define GLANCE_PUT(e_, sk_, t_, meta_, ps_)                                     \
    do {                                                                        \
        const int pe = (e_);                                                    \
        const bool pmine = (pe & 31) == lane;                                   \
        const int pslot = pe >> 5;                                              \
        const uint32_t psk = (sk_), pmeta = (meta_);                            \
        const unsigned long long ptw = (t_);                                    \
        const float pps = (ps_);                                                \
        GLANCE_SLOTS(GLANCE_PUT_OP)                                             \
    } while (0)
    auto tie_word = [](int depth, unsigned long long key) {
        return ((unsigned long long)(15 - depth) << 60) | (~key & 0x0fffffffffffffffull);
    };
    if (lane == 0) {
        n_token[0] = root_tok; n_parent[0] = -1; n_depth[0] = 0; n_rank[0] = 0; n_score[0] = 0.f;
    }
    if (lane < W) n_anc[lane] = (lane == 0) ? 1ull : 0ull;
    int nc = 1, fc = 0;                                  // node / frontier counts: the same in every lane
    if (L >= 1 && N > 1) {
        GLANCE_PUT(0, float_key(__fadd_rn(0.f, s_lp[0])), tie_word(1, 0ull), 1u, 0.f);
        fc = 1;
    }

    int live = fc;                                       // entries that are not empty slots
    while (live > 0 && nc < N) {
        // this lane's best entry
        uint32_t bsk = 0u;
        unsigned long long bt = 0ull;
        int bu = -1;
#define GLANCE_BEST_OP(u, sk, tw, me, ps) \
        if (u * 32 + lane < fc && (bu < 0 || sk > bsk || (sk == bsk && tw > bt))) { bsk = sk; bt = tw; bu = u; }
        GLANCE_SLOTS(GLANCE_BEST_OP)
        // warp arg-best: hardware max over the score image, then (rarely) over the halves of the tie word
        const uint32_t m1 = __reduce_max_sync(0xffffffffu, bu >= 0 ? bsk : 0u);
        uint32_t cand = __ballot_sync(0xffffffffu, bu >= 0 && bsk == m1);
        if (__popc(cand) > 1) {
            const bool in = (cand >> lane) & 1u;
            const uint32_t m2 = __reduce_max_sync(0xffffffffu, in ? (uint32_t)(bt >> 32) : 0u);
            cand = __ballot_sync(0xffffffffu, in && (uint32_t)(bt >> 32) == m2);
            if (__popc(cand) > 1) {
                const bool in2 = (cand >> lane) & 1u;
                const uint32_t m3 = __reduce_max_sync(0xffffffffu, in2 ? (uint32_t)bt : 0u);
                cand = __ballot_sync(0xffffffffu, in2 && (uint32_t)bt == m3);
            }
        }
        // (score, depth, key) identifies a candidate uniquely: exactly one lane is left; everybody takes its entry
        const int wl = __ffs(cand) - 1;
        uint32_t bmeta = 0u;
        float bps = 0.f;
#define GLANCE_META_OP(u, sk, tw, me, ps) if (bu == u) { bmeta = me; bps = ps; }
        GLANCE_SLOTS(GLANCE_META_OP)
        bu = __shfl_sync(0xffffffffu, bu, wl);
        bsk = __shfl_sync(0xffffffffu, bsk, wl);
        bt = __shfl_sync(0xffffffffu, bt, wl);
        bmeta = __shfl_sync(0xffffffffu, bmeta, wl);
        bps = __shfl_sync(0xffffffffu, bps, wl);
        const int dpt = bmeta & 15, rk = (bmeta >> 4) & 15, par = (int)(bmeta >> 8);
        const float sc = key_float(bsk);
        const unsigned long long key = ~bt & 0x0fffffffffffffffull;
        const int i = nc++;
        if (lane == 0) {
            n_token[i] = s_id[(dpt - 1) * k + rk];
            n_parent[i] = par; n_depth[i] = dpt; n_rank[i] = rk; n_score[i] = sc;
        }
        if (lane < W) {                                  // lane w owns word w of every node's mask
            unsigned long long aw = n_anc[par * W + lane];
            if ((i >> 6) == lane) aw |= 1ull << (i & 63);
            n_anc[i * W + lane] = aw;
        }
        // the child takes the popped entry's slot (or the slot goes empty: key 0 loses against every real entry); the
        // next sibling is appended -- the frontier grows by at most one entry per pop and nothing has to be moved
        const int bi = bu * 32 + wl;
        if (dpt < L) {
            GLANCE_PUT(bi, float_key(__fadd_rn(sc, s_lp[dpt * k])), tie_word(dpt + 1, key), (uint32_t)(dpt + 1) | ((uint32_t)i << 8), sc);
        } else {
            GLANCE_PUT(bi, 0u, 0ull, 0u, 0.f);
            --live;
        }
        if (rk + 1 < k) {
            GLANCE_PUT(fc, float_key(__fadd_rn(bps, s_lp[(dpt - 1) * k + rk + 1])), tie_word(dpt, key + (1ull << (4 * (15 - dpt)))), (uint32_t)dpt | ((uint32_t)(rk + 1) << 4) | ((uint32_t)par << 8), bps);
            ++fc;
            ++live;
        }
    }
#undef GLANCE_SLOTS
#undef GLANCE_PUT_OP
#undef GLANCE_PUT
#undef GLANCE_BEST_OP
#undef GLANCE_META_OP
    __syncwarp();
    if (lane == 0) out.n_nodes[s] = nc;
    int32_t *token = out.token + (size_t)s * N, *parent = out.parent + (size_t)s * N;
    int32_t *depth = out.depth + (size_t)s * N, *rank = out.rank + (size_t)s * N;
    float *score = out.score + (size_t)s * N;
    uint64_t *anc = out.anc + (size_t)s * N * W;
    for (int i = lane; i < N; i += 32) {
        // padding rows: never entered by the walk, visible to themselves only
        const bool real = i < nc;
        token[i] = real ? n_token[i] : 0;
        parent[i] = real ? n_parent[i] : -1;
        depth[i] = real ? n_depth[i] : 0;
        rank[i] = real ? n_rank[i] : 0;
        score[i] = real ? n_score[i] : 0.f;
        for (int w = 0; w < W; ++w)
            anc[(size_t)i * W + w] = real ? n_anc[i * W + w] : (((i >> 6) == w) ? (1ull << (i & 63)) : 0ull);
    }
}

void launch_build_tree(int batch, int N, int L, int k, const int32_t *root, const int32_t *ids, const float *lp,
                       const glance_tree &out, cudaStream_t st) {
    build_tree_kernel<<<batch, 32, 0, st>>>(N, L, k, root, ids, lp, out);
}

// ------------------------------------------------------------------------------------------
// Walk + commit in one kernel.
//
// Grid (batch, n_layers * 2 * Hkv).  Every block repeats the (tiny) walk, then compacts its own
// (layer, K|V, kv head) slice: cache row P + path[d] -> row P + d for d = 1..a.  Destination row P + d
// can be the source row of a later step (path is strictly increasing with path[d] >= d), so a block
// loads all its sources before it stores anything.  The last block of a sequence to finish publishes
// the outputs and advances the sequence state, so no block reads seq_len after it changed.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) walk_commit_kernel(WalkCommit p) {
    __shared__ int sh_path[kMaxBlock + 1];
    __shared__ int sh_a, sh_root, sh_last;
    const int s = blockIdx.x;
    const int P = p.seq_len[s];
    const int L = p.B - 1;

    // the walk's three small arrays are fetched once, coalesced, instead of one dependent global load per step
    __shared__ int sh_am[kMaxTreeN], sh_tok[kMaxTreeN], sh_par[kMaxTreeN];
    if (p.argmax) {
        for (int i = threadIdx.x; i < p.N; i += blockDim.x) {
            sh_am[i] = p.argmax[(size_t)s * p.N + i];
            sh_tok[i] = p.token[(size_t)s * p.N + i];
            sh_par[i] = p.parent[(size_t)s * p.N + i];
        }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        if (p.argmax) {
            const int *am = sh_am, *tok = sh_tok, *par = sh_par;
            int nn = p.n_nodes[s];
            nn = nn < 1 ? 1 : (nn > p.N ? p.N : nn);
            int v = 0, a = 0, t = am[0];
            if (lane == 0) sh_path[0] = 0;
            while (a < L) {
                int found = 1 << 30;
                for (int c = 1 + lane; c < nn; c += 32)
                    if (par[c] == v && tok[c] == t && c < found) found = c;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) found = min(found, __shfl_xor_sync(0xffffffffu, found, o));
                if (found == (1 << 30)) break;
                v = found;
                ++a;
                if (lane == 0) sh_path[a] = v;
                t = am[v];
            }
            if (lane == 0) { sh_a = a; sh_root = t; }
        } else if (lane == 0) {
            int len = p.forced_len[s];
            len = len < 1 ? 1 : (len > p.B ? p.B : len);
            int prev = -1;
            bool ok = true;
            for (int d = 0; d < len; ++d) {
                int v = p.forced_path[(size_t)s * p.B + d];
                if (v <= prev || v >= p.N || (d == 0 && v != 0)) ok = false;
                prev = v;
                sh_path[d] = ok ? v : d;
            }
            if (!ok) set_status(p.status, GLANCE_E_BOUNDS);
            sh_a = len - 1;
            sh_root = p.forced_root[s];
        }
    }
    __syncthreads();
    const int a = sh_a;

    // compaction of this block's slice
    const int slice = blockIdx.y;                       // (layer, kv, head)
    const int per_layer = 2 * p.geom.n_kv_heads;
    const int layer = slice / per_layer, kv = (slice % per_layer) / p.geom.n_kv_heads;
    const int head = slice % p.geom.n_kv_heads;
    bf16 *base = p.kv_pool + (size_t)layer * p.geom.layer_stride();
    const int chunks = p.geom.head_dim * 2 / 16;        // 16-byte chunks per row
    const int items = a * chunks;
    const int32_t *pt = p.page_table + (size_t)s * p.geom.max_pages_per_seq;
    for (int it0 = 0; it0 < items; it0 += blockDim.x) {
        const int it = it0 + threadIdx.x;
        int4 val;
        int4 *dst = nullptr;
        if (it < items) {
            const int d = 1 + it / chunks, c = it % chunks;
            const int src_pos = P + sh_path[d], dst_pos = P + d;
            const int sp = src_pos / kPage, dp = dst_pos / kPage;
            if (sp < p.geom.max_pages_per_seq && dp < p.geom.max_pages_per_seq) {
                const int spage = pt[sp], dpage = pt[dp];
                if (spage >= 0 && spage < p.geom.n_pages && dpage >= 0 && dpage < p.geom.n_pages) {
                    const int4 *src = reinterpret_cast<const int4 *>(base + p.geom.row(spage, kv, head, src_pos % kPage)) + c;
                    dst = reinterpret_cast<int4 *>(base + p.geom.row(dpage, kv, head, dst_pos % kPage)) + c;
                    val = *src;
                }
            }
            if (!dst) set_status(p.status, GLANCE_E_BOUNDS);
        }
        __syncthreads();                                // all sources of this batch are in registers
        if (dst) *dst = val;
        __syncthreads();
    }

    // features of the accepted path (every tap slice): hidden[path[i]] -> feat[i], in 16-byte pieces shared out over
    // all blocks of the sequence (nothing reads feat before the next draft pass)
    {
        const int CH = p.H >> 3;                        // H is a multiple of 64
        const int per_tap = (a + 1) * CH;
        const int total = p.n_taps * per_tap;
        for (int it = blockIdx.y * blockDim.x + threadIdx.x; it < total; it += gridDim.y * blockDim.x) {
            const int tap = it / per_tap, rem = it - tap * per_tap;
            const int i = rem / CH, c = rem - i * CH;
            const int4 *src = reinterpret_cast<const int4 *>(p.hidden + ((size_t)tap * p.batch * p.N + (size_t)s * p.N + sh_path[i]) * p.H) + c;
            int4 *dst = reinterpret_cast<int4 *>(p.feat + ((size_t)tap * p.batch * p.B + (size_t)s * p.B + i) * p.H) + c;
            *dst = *src;
        }
    }

    // last block of the sequence publishes the outcome
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) sh_last = (atomicAdd(&p.counters[s], 1) == (int)gridDim.y - 1);
    __syncthreads();
    if (!sh_last) return;
    if (threadIdx.x == 0) {
        if (p.accept_len) p.accept_len[s] = a;
        for (int d = 0; d < p.B; ++d) {
            if (p.path) p.path[(size_t)s * p.B + d] = d <= a ? sh_path[d] : -1;
            if (p.out_tokens) {
                int t = -1;
                if (d < a) t = p.token ? p.token[(size_t)s * p.N + sh_path[d + 1]] : -1;
                else if (d == a) t = sh_root;
                p.out_tokens[(size_t)s * p.B + d] = t;
            }
        }
        p.feat_count[s] = a + 1;
        p.seq_len[s] = P + a + 1;
        p.root[s] = sh_root;
        p.counters[s] = 0;
    }
}

void launch_walk_commit(const WalkCommit &p, cudaStream_t st) {
    dim3 grid(p.batch, p.n_layers * 2 * p.geom.n_kv_heads);
    walk_commit_kernel<<<grid, 256, 0, st>>>(p);
}

}  // namespace glance
