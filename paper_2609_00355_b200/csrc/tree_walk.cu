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

__global__ void __launch_bounds__(32) build_tree_kernel(int N, int L, int k, const int32_t *root, const int32_t *ids,
                                                        const float *lp, glance_tree out) {
    constexpr int CAP = kMaxTreeN + 4;
    __shared__ float f_score[CAP];
    __shared__ int f_depth[CAP], f_rank[CAP], f_parent[CAP];
    __shared__ unsigned long long f_key[CAP];
    __shared__ float n_score[kMaxTreeN];
    __shared__ int n_count, f_count;

    const int s = blockIdx.x, lane = threadIdx.x;
    const int W = (N + 63) >> 6;
    const int32_t *sid = ids + (size_t)s * L * k;
    const float *slp = lp + (size_t)s * L * k;
    int32_t *token = out.token + (size_t)s * N, *parent = out.parent + (size_t)s * N;
    int32_t *depth = out.depth + (size_t)s * N, *rank = out.rank + (size_t)s * N;
    float *score = out.score + (size_t)s * N;
    uint64_t *anc = out.anc + (size_t)s * N * W;

    if (lane == 0) {
        token[0] = root[s]; parent[0] = -1; depth[0] = 0; rank[0] = 0; score[0] = 0.f;
        n_score[0] = 0.f;
        n_count = 1;
        f_count = 0;
        if (L >= 1 && N > 1) {
            f_score[0] = __fadd_rn(0.f, slp[0]);
            f_depth[0] = 1; f_rank[0] = 0; f_parent[0] = 0; f_key[0] = 0ull;
            f_count = 1;
        }
    }
    if (lane < W) anc[lane] = (lane == 0) ? 1ull : 0ull;
    __syncwarp();

    while (true) {
        const int fc = f_count, nc = n_count;
        if (fc == 0 || nc >= N) break;
        // warp arg-best over the frontier
        Cand best;
        best.score = -INFINITY; best.depth = 1 << 30; best.key = ~0ull;
        int bi = -1;
        for (int e = lane; e < fc; e += 32) {
            Cand c; c.score = f_score[e]; c.depth = f_depth[e]; c.key = f_key[e];
            if (bi < 0 || cand_before(c, best)) { best = c; bi = e; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            Cand c;
            c.score = __shfl_xor_sync(0xffffffffu, best.score, o);
            c.depth = __shfl_xor_sync(0xffffffffu, best.depth, o);
            c.key = __shfl_xor_sync(0xffffffffu, best.key, o);
            const int ci = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ci >= 0 && (bi < 0 || cand_before(c, best))) { best = c; bi = ci; }
        }
        // (score, depth, key) identifies a candidate uniquely, so every lane now agrees on bi
        const int i = nc;
        const int dpt = f_depth[bi], rk = f_rank[bi], par = f_parent[bi];
        const float sc = f_score[bi];
        const unsigned long long key = f_key[bi];
        __syncwarp();
        if (lane < W) {
            uint64_t w = anc[(size_t)par * W + lane];
            if ((i >> 6) == lane) w |= 1ull << (i & 63);
            anc[(size_t)i * W + lane] = w;
        }
        if (lane == 0) {
            token[i] = sid[(dpt - 1) * k + rk];
            parent[i] = par; depth[i] = dpt; rank[i] = rk; score[i] = sc;
            n_score[i] = sc;
            n_count = nc + 1;
            // remove the popped entry (swap with the last), then push child and sibling
            int cnt = fc - 1;
            if (bi != cnt) {
                f_score[bi] = f_score[cnt]; f_depth[bi] = f_depth[cnt]; f_rank[bi] = f_rank[cnt];
                f_parent[bi] = f_parent[cnt]; f_key[bi] = f_key[cnt];
            }
            if (dpt < L) {
                f_score[cnt] = __fadd_rn(sc, slp[dpt * k + 0]);
                f_depth[cnt] = dpt + 1; f_rank[cnt] = 0; f_parent[cnt] = i; f_key[cnt] = key;
                ++cnt;
            }
            if (rk + 1 < k) {
                f_score[cnt] = __fadd_rn(n_score[par], slp[(dpt - 1) * k + rk + 1]);
                f_depth[cnt] = dpt; f_rank[cnt] = rk + 1; f_parent[cnt] = par;
                f_key[cnt] = key + (1ull << (4 * (15 - dpt)));
                ++cnt;
            }
            f_count = cnt;
        }
        __syncwarp();
    }
    __syncwarp();
    const int nc = n_count;
    if (lane == 0) out.n_nodes[s] = nc;
    // padding rows: never entered by the walk, visible to themselves only
    for (int i = nc + lane; i < N; i += 32) {
        token[i] = 0; parent[i] = -1; depth[i] = 0; rank[i] = 0; score[i] = 0.f;
        for (int w = 0; w < W; ++w) anc[(size_t)i * W + w] = ((i >> 6) == w) ? (1ull << (i & 63)) : 0ull;
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

    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        if (p.argmax) {
            const int32_t *am = p.argmax + (size_t)s * p.N;
            const int32_t *tok = p.token + (size_t)s * p.N, *par = p.parent + (size_t)s * p.N;
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

    // last block of the sequence publishes the outcome
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) sh_last = (atomicAdd(&p.counters[s], 1) == (int)gridDim.y - 1);
    __syncthreads();
    if (!sh_last) return;
    for (int i = 0; i <= a; ++i) {
        const bf16 *src = p.hidden + ((size_t)s * p.N + sh_path[i]) * p.H;
        bf16 *dst = p.feat + ((size_t)s * p.B + i) * p.H;
        for (int c = threadIdx.x; c < p.H; c += blockDim.x) dst[c] = src[c];
    }
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
