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

// Everything the loop touches lives in shared memory (candidate tables, node arrays, ancestor masks): an
// iteration is a handful of shared-memory accesses and one warp reduction; the tree is written out once at the end.
__global__ void __launch_bounds__(32) build_tree_kernel(int N, int L, int k, const int32_t *root, const int32_t *ids,
                                                        const float *lp, glance_tree out) {
    constexpr int CAP = kMaxTreeN + 4;
    __shared__ float f_score[CAP];
    __shared__ int f_depth[CAP], f_rank[CAP], f_parent[CAP];
    __shared__ unsigned long long f_key[CAP];
    __shared__ uint32_t f_sk[CAP];                   // order-preserving image of f_score
    __shared__ unsigned long long f_t[CAP];          // tie word: (15 - depth) << 60 | ~key
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

    auto tie_word = [](int depth, unsigned long long key) {
        return ((unsigned long long)(15 - depth) << 60) | (~key & 0x0fffffffffffffffull);
    };
    int nc = 1, fc = 0;                                  // node / frontier counts: the same in every lane
    if (L >= 1 && N > 1) fc = 1;
    if (lane == 0) {
        n_token[0] = root_tok; n_parent[0] = -1; n_depth[0] = 0; n_rank[0] = 0; n_score[0] = 0.f;
        if (fc) {
            const float sc0 = __fadd_rn(0.f, s_lp[0]);
            f_score[0] = sc0; f_sk[0] = float_key(sc0);
            f_depth[0] = 1; f_rank[0] = 0; f_parent[0] = 0; f_key[0] = 0ull; f_t[0] = tie_word(1, 0ull);
        }
    }
    if (lane < W) n_anc[lane] = (lane == 0) ? 1ull : 0ull;
    __syncwarp();

    // The order (score desc, depth asc, key asc) as integers: a 32-bit order-preserving image of the score and a
    // 64-bit tie word (15 - depth in the top four bits, the complemented 60-bit path key below); larger wins.
    while (fc > 0 && nc < N) {
        uint32_t bsk = 0;
        unsigned long long bt = 0ull;
        int bi = -1;
        for (int e = lane; e < fc; e += 32) {
            const uint32_t sk = f_sk[e];
            const unsigned long long t = f_t[e];
            if (bi < 0 || sk > bsk || (sk == bsk && t > bt)) { bsk = sk; bt = t; bi = e; }
        }
        // warp arg-best: hardware max over the score image, then (rarely) over the halves of the tie word
        const uint32_t m1 = __reduce_max_sync(0xffffffffu, bi >= 0 ? bsk : 0u);
        uint32_t live = __ballot_sync(0xffffffffu, bi >= 0 && bsk == m1);
        if (__popc(live) > 1) {
            const bool in = (live >> lane) & 1u;
            const uint32_t m2 = __reduce_max_sync(0xffffffffu, in ? (uint32_t)(bt >> 32) : 0u);
            live = __ballot_sync(0xffffffffu, in && (uint32_t)(bt >> 32) == m2);
            if (__popc(live) > 1) {
                const bool in2 = (live >> lane) & 1u;
                const uint32_t m3 = __reduce_max_sync(0xffffffffu, in2 ? (uint32_t)bt : 0u);
                live = __ballot_sync(0xffffffffu, in2 && (uint32_t)bt == m3);
            }
        }
        // (score, depth, key) identifies a candidate uniquely: exactly one lane is left
        bi = __shfl_sync(0xffffffffu, bi, __ffs(live) - 1);
        const int i = nc;
        const int dpt = f_depth[bi], rk = f_rank[bi], par = f_parent[bi];
        const float sc = f_score[bi];
        const unsigned long long key = f_key[bi];
        // the popped entry is replaced by the last one; the child and the next sibling are appended
        const int last = fc - 1;
        const bool has_child = dpt < L, has_sib = rk + 1 < k;
        float mv_score = 0.f; int mv_depth = 0, mv_rank = 0, mv_parent = 0; unsigned long long mv_key = 0ull, mv_t = 0ull;
        uint32_t mv_sk = 0u;
        if (lane == 3 && bi != last) {
            mv_score = f_score[last]; mv_depth = f_depth[last]; mv_rank = f_rank[last];
            mv_parent = f_parent[last]; mv_key = f_key[last]; mv_sk = f_sk[last]; mv_t = f_t[last];
        }
        unsigned long long aw = 0ull;
        if (lane < W) {
            aw = n_anc[par * W + lane];
            if ((i >> 6) == lane) aw |= 1ull << (i & 63);
        }
        const float par_score = n_score[par];
        __syncwarp();                                    // all reads of the old frontier are done
        if (lane < W) n_anc[i * W + lane] = aw;
        if (lane == 0) {
            n_token[i] = s_id[(dpt - 1) * k + rk];
            n_parent[i] = par; n_depth[i] = dpt; n_rank[i] = rk; n_score[i] = sc;
        } else if (lane == 1 && has_child) {
            const float cs = __fadd_rn(sc, s_lp[dpt * k + 0]);
            f_score[last] = cs; f_sk[last] = float_key(cs);
            f_depth[last] = dpt + 1; f_rank[last] = 0; f_parent[last] = i; f_key[last] = key; f_t[last] = tie_word(dpt + 1, key);
        } else if (lane == 2 && has_sib) {
            const int at = last + (has_child ? 1 : 0);
            const float ss = __fadd_rn(par_score, s_lp[(dpt - 1) * k + rk + 1]);
            const unsigned long long sk2 = key + (1ull << (4 * (15 - dpt)));
            f_score[at] = ss; f_sk[at] = float_key(ss);
            f_depth[at] = dpt; f_rank[at] = rk + 1; f_parent[at] = par;
            f_key[at] = sk2; f_t[at] = tie_word(dpt, sk2);
        } else if (lane == 3 && bi != last) {
            f_score[bi] = mv_score; f_depth[bi] = mv_depth; f_rank[bi] = mv_rank; f_parent[bi] = mv_parent; f_key[bi] = mv_key;
            f_sk[bi] = mv_sk; f_t[bi] = mv_t;
        }
        nc = nc + 1;
        fc = last + (has_child ? 1 : 0) + (has_sib ? 1 : 0);
        __syncwarp();
    }
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
