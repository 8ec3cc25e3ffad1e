"""CPU oracle for one GLANCE speculative decoding round.  TEST INFRASTRUCTURE ONLY.

Plain, slow, fp32 PyTorch-CPU / numpy / pure-Python statement of what the round
computes, written from the paper (Section 3, Definition 1, Theorem 1, Algorithm 1).
It shares no code with the CUDA library and must never be imported by it; only
tests, the smoke check and the benchmark's cpu-baseline leg may call it.

Two groups of functions:

  (I) plain definitions the method must reproduce exactly
      * greedy_ar_cachefree   -- Section 3.1: Y_k = argmax p(. | x o b o Y_1:k-1), one full
                                 causal forward per token, no cache
      * accepted_length_bruteforce -- Definition 1: A(S) = max{k : Y_1:j in S for all j <= k}
      * chain_row             -- Definition 1: row of node y_1:d is p(. | x o b o y_1:d),
                                 recomputed as a plain causal chain
      * build_tree_bruteforce -- Algorithm 1 line 2: enumerate every prefix, sort, keep the best

 (II) the round step by step, in the order of Algorithm 1
      prefill -> draft_block -> topk_logprobs -> build_tree -> verify_tree -> walk -> commit

Readings of points the paper leaves open:
  * the verify pass has N rows including the root; the paper's budget is N-1
  * horizon L = B-1; block slot 0 holds the root, slot j predicts offset j (no shift)
  * the one-layer head attends to [context features ; block] with one set of W_k/W_v;
    context features are the target's residual stream after the last layer, before the
    final norm, for committed positions only; the root enters as its embedding
  * the multi-layer head (Section 3.2: five layers, keys/values from five kept target layers): head layer i is
    one such layer with its own weights whose context keys/values are projections of the residual stream after
    target layer taps[i]; the block rows flow through the head layers in order
  * q_j is the full-vocabulary softmax; candidates are restricted to per-slot top-k
  * ties: argmax/top-k prefer the lowest id; tree order is (score desc, depth asc,
    path key asc); node index = position in that order
  * 1-D rotary positions (context 0..P-1, node at P+depth, block slot j at P+j),
    rotate-half pairing (i, i+d/2)

Pins (tests/test_oracle_*.py): losslessness against greedy_ar_cachefree for best-first,
random, chain and single-node trees; accepted length against brute-force membership;
verify rows against chain_row; chain mask = causal; best-first = brute-force sort;
attention against torch SDPA; top-k / lse against torch.topk / logsumexp; rotary
relative-position identity; KV state after rounds = fresh prefill.
sampling mode (Limitations section): Philox known-answer vectors, uniforms strictly inside (0,1), draw frequencies
against the softmax, and tree rounds against plain ancestral sampling with the same noise field.
multi-layer head: taps against truncated cache-free forwards, the stack against repeated decoder_layer calls,
the one-tap case bit-identical to the one-layer head, head state after rounds = fresh prefill for every layer.
draft_block (the reading of Section 3.2 stated above; the paper prints no worked example of the head):
equality with decoder_layer under an all-ones mask, the identity-layer closed form (W_o = W_down = 0), the
single-key closed form (B = 1, no context) written out in float64, invariance under a permutation of the
context rows.
"""
from __future__ import annotations

import heapq
import itertools
import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

F32 = torch.float32


# ----------------------------------------------------------------------------------------------
# model pieces (RMSNorm, rotary, GQA attention, SwiGLU) -- the decoder named by the configs
# ----------------------------------------------------------------------------------------------

@dataclass(frozen=True)
class Shape:
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    rms_eps: float = 1e-6
    rope_theta: float = 1e6
    head_taps: Tuple[int, ...] = ()      # () = one head layer fed by the last target layer; else one tap per head layer

    @staticmethod
    def of(cfg) -> "Shape":
        return Shape(cfg.n_layers, cfg.hidden, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.ffn,
                     cfg.vocab, cfg.rms_eps, cfg.rope_theta, tuple(getattr(cfg, "head_taps", ()) or ()))

    @property
    def taps(self) -> Tuple[int, ...]:
        """Target layer (0-based) whose output feeds head layer i."""
        return self.head_taps if self.head_taps else (self.n_layers - 1,)


def widen(w):
    """bf16 weight bits -> fp32 values (exact)."""
    if isinstance(w, dict):
        return {k: widen(v) for k, v in w.items()}
    if isinstance(w, list):
        return [widen(v) for v in w]
    return w.detach().to("cpu").to(F32)


def rmsnorm(x: torch.Tensor, g: torch.Tensor, eps: float) -> torch.Tensor:
    return x * torch.rsqrt((x * x).mean(dim=-1, keepdim=True) + eps) * g


def rope(x: torch.Tensor, pos: torch.Tensor, theta: float) -> torch.Tensor:
    """x [n, heads, d]; rotates pair (i, i + d/2) by angle pos * theta^(-2i/d)."""
    d = x.shape[-1]
    half = d // 2
    inv = torch.tensor([theta ** (-(2.0 * i) / d) for i in range(half)], dtype=torch.float64)
    ang = pos.to(torch.float64)[:, None] * inv[None, :]
    cos = ang.cos().to(F32)[:, None, :]
    sin = ang.sin().to(F32)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


def attention(q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, mask: torch.Tensor) -> torch.Tensor:
    """q [n,Hq,d], K/V [m,Hkv,d], mask [n,m] bool (True = visible) -> [n,Hq,d].

    softmax(q k^T / sqrt(d)) v with q head h reading kv head h // (Hq/Hkv).
    """
    n, Hq, d = q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    out = torch.empty_like(q)
    scale = 1.0 / math.sqrt(d)
    for h in range(Hq):
        kv = h // G
        s = (q[:, h, :] @ K[:, kv, :].T) * scale
        s = s.masked_fill(~mask, float("-inf"))
        p = torch.softmax(s, dim=-1)
        out[:, h, :] = p @ V[:, kv, :]
    return out


def split_qkv(sh: Shape, y: torch.Tensor):
    n = y.shape[0]
    qd = sh.n_q_heads * sh.head_dim
    kd = sh.n_kv_heads * sh.head_dim
    q = y[:, :qd].reshape(n, sh.n_q_heads, sh.head_dim)
    k = y[:, qd:qd + kd].reshape(n, sh.n_kv_heads, sh.head_dim)
    v = y[:, qd + kd:].reshape(n, sh.n_kv_heads, sh.head_dim)
    return q, k, v


def mlp(sh: Shape, h2: torch.Tensor, wgu: torch.Tensor, wd: torch.Tensor) -> torch.Tensor:
    gu = h2 @ wgu.T
    g, u = gu[:, :sh.ffn], gu[:, sh.ffn:]
    return (torch.nn.functional.silu(g) * u) @ wd.T


def decoder_layer(sh: Shape, lw: dict, x: torch.Tensor, pos: torch.Tensor, Kc: torch.Tensor, Vc: torch.Tensor,
                  rows: torch.Tensor, mask: torch.Tensor) -> torch.Tensor:
    """One target layer over n new rows.

    K/V of the new rows are written into cache rows `rows` of Kc/Vc ([cap,Hkv,d]); the
    queries then attend to cache rows 0..mask.shape[1]-1 under `mask`.
    """
    h1 = rmsnorm(x, lw["ln1"], sh.rms_eps)
    q, k, v = split_qkv(sh, h1 @ lw["wqkv"].T)
    q = rope(q, pos, sh.rope_theta)
    k = rope(k, pos, sh.rope_theta)
    Kc[rows] = k
    Vc[rows] = v
    m = mask.shape[1]
    o = attention(q, Kc[:m], Vc[:m], mask)
    x = x + o.reshape(x.shape[0], -1) @ lw["wo"].T
    h2 = rmsnorm(x, lw["ln2"], sh.rms_eps)
    return x + mlp(sh, h2, lw["wgu"], lw["wd"])


def argmax_lowest(logits: torch.Tensor) -> np.ndarray:
    """Row-wise argmax, ties to the lowest id."""
    mx = logits.max(dim=-1, keepdim=True).values
    first = (logits == mx).to(torch.int8).argmax(dim=-1)
    return first.numpy().astype(np.int32)


# ----------------------------------------------------------------------------------------------
# (I) plain definitions
# ----------------------------------------------------------------------------------------------

def full_causal_forward(sh: Shape, tw: dict, x_in: torch.Tensor):
    """Causal forward of a whole sequence of input embeddings [T,H] with no cache.

    Returns (logits [T,V], features [T,H]); feature = residual stream after the last
    layer, before the final norm.
    """
    T = x_in.shape[0]
    pos = torch.arange(T)
    mask = torch.tril(torch.ones(T, T, dtype=torch.bool))
    x = x_in.clone()
    for lw in tw["layers"]:
        Kc = torch.zeros(T, sh.n_kv_heads, sh.head_dim)
        Vc = torch.zeros(T, sh.n_kv_heads, sh.head_dim)
        x = decoder_layer(sh, lw, x, pos, Kc, Vc, pos, mask)
    logits = rmsnorm(x, tw["final_norm"], sh.rms_eps) @ tw["lm_head"].T
    return logits, x


def context_embeddings(tw: dict, image_embeds: torch.Tensor, text_ids) -> torch.Tensor:
    """Input rows of the multimodal prefix: image embeddings first, then E[text id]."""
    ids = torch.as_tensor(np.asarray(text_ids), dtype=torch.long)
    return torch.cat([image_embeds.to(F32), tw["embed"][ids]], dim=0)


def greedy_ar_cachefree(sh: Shape, tw: dict, ctx_embeds: torch.Tensor, n_new: int):
    """Plain greedy decoding (Section 3.1): one full causal forward per emitted token.

    Returns (tokens [n_new], margins [n_new]) where tokens[0] is the first token after the
    context (the first round's root) and margins are the top-1 minus top-2 logit gaps.
    """
    x = ctx_embeds.clone()
    toks, margins = [], []
    for _ in range(n_new):
        logits, _ = full_causal_forward(sh, tw, x)
        last = logits[-1]
        t = int(argmax_lowest(last[None, :])[0])
        top2 = torch.topk(last, 2).values
        margins.append(float(top2[0] - top2[1]))
        toks.append(t)
        x = torch.cat([x, tw["embed"][t][None, :]], dim=0)
    return toks, margins


def tree_paths(tree: "Tree") -> Dict[Tuple[int, ...], int]:
    """The candidate set S as {token string after the root: node index}."""
    out: Dict[Tuple[int, ...], int] = {}
    for i in range(1, tree.n_nodes):
        s: List[int] = []
        v = i
        while v != 0:
            s.append(int(tree.token[v]))
            v = int(tree.parent[v])
        out[tuple(reversed(s))] = i
    return out


def accepted_length_bruteforce(tree: "Tree", Y: Sequence[int]) -> int:
    """Definition 1: A(S) = max{k >= 0 : Y_1:j in S for every j <= k}; Y = greedy continuation after the root."""
    S = tree_paths(tree)
    k = 0
    while k < len(Y) and tuple(int(t) for t in Y[:k + 1]) in S:
        k += 1
    return k


def chain_row(sh: Shape, tw: dict, ctx_embeds: torch.Tensor, root: int, string: Sequence[int]):
    """Definition 1: logits p(. | x o b o y_1:d) by a plain causal forward of the whole chain."""
    toks = [int(root)] + [int(t) for t in string]
    x = torch.cat([ctx_embeds, tw["embed"][torch.tensor(toks, dtype=torch.long)]], dim=0)
    logits, feats = full_causal_forward(sh, tw, x)
    return logits[-1], feats[-1]


# ----------------------------------------------------------------------------------------------
# candidate tree (Definition 1, Algorithm 1 lines 2-3)
# ----------------------------------------------------------------------------------------------

@dataclass
class Tree:
    token: np.ndarray            # [N] int32; token[0] = root b
    parent: np.ndarray           # [N] int32; -1 for the root and for padding rows
    depth: np.ndarray            # [N] int32
    rank: np.ndarray             # [N] int32; rank of the node's token within its depth's top-k
    score: np.ndarray            # [N] float32; sum of log q along the path (left-to-right fp32 adds)
    anc: np.ndarray              # [N][ceil(N/64)] uint64; bit j of row i = node j is i or an ancestor of i
    n_nodes: int                 # real nodes including the root; rows beyond are padding

    @property
    def N(self) -> int:
        return int(self.token.shape[0])


def ancestor_mask(parent: np.ndarray, n_nodes: int, N: int) -> np.ndarray:
    """anc[i] = {i} union anc[parent[i]]; padding rows see only themselves.  Bit j -> word j>>6, bit j&63."""
    W = (N + 63) // 64
    anc = np.zeros((N, W), dtype=np.uint64)
    for i in range(N):
        if i < n_nodes and parent[i] >= 0:
            anc[i] = anc[int(parent[i])]
        anc[i, i >> 6] |= np.uint64(1) << np.uint64(i & 63)
    return anc


def tree_from_arrays(token, parent, depth, N: Optional[int] = None, rank=None, score=None) -> Tree:
    """Wrap caller-given (token, parent, depth) of n real nodes into a padded Tree of N rows."""
    n = len(token)
    N = n if N is None else N
    tk = np.zeros(N, dtype=np.int32); tk[:n] = token
    pa = np.full(N, -1, dtype=np.int32); pa[:n] = parent
    de = np.zeros(N, dtype=np.int32); de[:n] = depth
    rk = np.zeros(N, dtype=np.int32)
    sc = np.zeros(N, dtype=np.float32)
    if rank is not None:
        rk[:n] = rank
    if score is not None:
        sc[:n] = score
    return Tree(tk, pa, de, rk, sc, ancestor_mask(pa, n, N), n)


def chain_tree(root: int, tokens: Sequence[int], N: Optional[int] = None) -> Tree:
    n = 1 + len(tokens)
    return tree_from_arrays([root] + list(tokens), [-1] + list(range(n - 1)), list(range(n)), N)


def _path_key(ranks: Sequence[int]) -> int:
    key = 0
    for i, r in enumerate(ranks, start=1):
        key += int(r) * (16 ** (15 - i))
    return key


def build_tree(root: int, ids: np.ndarray, lp: np.ndarray, N: int) -> Tree:
    """Algorithm 1 line 2 by best-first search.

    ids/lp [L][k]: per-offset top-k token ids and fp32 log-probabilities (row j-1 = offset j,
    lp non-increasing along a row).  Keeps the M = min(N-1, sum_l k^l) prefixes of highest
    score = fl32(score[parent] + lp[depth][rank]) under the total order (score desc, depth
    asc, path key asc); node index = position in that order; node 0 = root.
    The frontier holds, for every kept node, its rank-0 child and its next-rank sibling:
    both score no higher than the node itself, so popping the best frontier entry
    enumerates the order exactly.
    """
    L, k = ids.shape
    lp = lp.astype(np.float32)
    token = np.zeros(N, dtype=np.int32); token[0] = root
    parent = np.full(N, -1, dtype=np.int32)
    depth = np.zeros(N, dtype=np.int32)
    rank = np.zeros(N, dtype=np.int32)
    score = np.zeros(N, dtype=np.float32)
    # entry: (-score, depth, path key, ranks, parent node)
    heap: List[tuple] = []
    if L >= 1 and N > 1:
        s0 = np.float32(np.float32(0.0) + lp[0][0])
        heapq.heappush(heap, (-float(s0), 1, _path_key((0,)), (0,), 0))
    n = 1
    while heap and n < N:
        negs, dpt, _, ranks, par = heapq.heappop(heap)
        i = n
        n += 1
        token[i] = ids[dpt - 1][ranks[-1]]
        parent[i] = par
        depth[i] = dpt
        rank[i] = ranks[-1]
        score[i] = np.float32(-negs)
        if dpt < L:
            cs = np.float32(score[i] + lp[dpt][0])
            cr = ranks + (0,)
            heapq.heappush(heap, (-float(cs), dpt + 1, _path_key(cr), cr, i))
        if ranks[-1] + 1 < k:
            ss = np.float32(score[par] + lp[dpt - 1][ranks[-1] + 1])
            sr = ranks[:-1] + (ranks[-1] + 1,)
            heapq.heappush(heap, (-float(ss), dpt, _path_key(sr), sr, par))
    return Tree(token, parent, depth, rank, score, ancestor_mask(parent, n, N), n)


def build_tree_bruteforce(root: int, ids: np.ndarray, lp: np.ndarray, N: int) -> Tree:
    """Algorithm 1 line 2 as written: score every prefix of every length, sort, keep the best N-1."""
    L, k = ids.shape
    lp = lp.astype(np.float32)
    cands = []
    for ell in range(1, L + 1):
        for ranks in itertools.product(range(k), repeat=ell):
            s = np.float32(0.0)
            for j, r in enumerate(ranks):
                s = np.float32(s + lp[j][r])
            cands.append((-float(s), ell, _path_key(ranks), ranks))
    cands.sort()
    kept = cands[:N - 1]
    index = {(): 0}
    token = np.zeros(N, dtype=np.int32); token[0] = root
    parent = np.full(N, -1, dtype=np.int32)
    depth = np.zeros(N, dtype=np.int32)
    rank = np.zeros(N, dtype=np.int32)
    score = np.zeros(N, dtype=np.float32)
    for i, (negs, ell, _, ranks) in enumerate(kept, start=1):
        index[ranks] = i
        token[i] = ids[ell - 1][ranks[-1]]
        parent[i] = index[ranks[:-1]]       # KeyError here would mean the kept set is not prefix-closed
        depth[i] = ell
        rank[i] = ranks[-1]
        score[i] = np.float32(-negs)
    n = len(kept) + 1
    return Tree(token, parent, depth, rank, score, ancestor_mask(parent, n, N), n)


def visibility(tree: Tree, P: int) -> torch.Tensor:
    """Packed-pass mask [N, P+N]: context fully visible, tree key j visible to row i iff anc[i] bit j."""
    N = tree.N
    m = torch.zeros(N, P + N, dtype=torch.bool)
    m[:, :P] = True
    for i in range(N):
        for j in range(N):
            if (int(tree.anc[i, j >> 6]) >> (j & 63)) & 1:
                m[i, P + j] = True
    return m


# ----------------------------------------------------------------------------------------------
# (II) the round, step by step
# ----------------------------------------------------------------------------------------------

@dataclass
class SeqState:
    """Logical (unpaged) state of one sequence: committed length P, pending root, caches."""
    P: int
    root: int
    K: List[torch.Tensor]        # per target layer [cap,Hkv,d]
    V: List[torch.Tensor]
    hK: torch.Tensor             # head context keys [cap,Hkv,d]
    hV: torch.Tensor
    feat: torch.Tensor           # [cap,H] target features of committed positions (tap of head layer 0)
    tokens: List[int] = field(default_factory=list)   # committed tokens after the context (for audits)
    # head layers 1.. of a multi-layer head (Section 3.2: five layers, one tapped target layer each)
    hK_more: List[torch.Tensor] = field(default_factory=list)
    hV_more: List[torch.Tensor] = field(default_factory=list)
    feat_more: List[torch.Tensor] = field(default_factory=list)


def head_layer(hw: dict, i: int) -> dict:
    """Weights of head layer i: layer 0 lives in the flat keys, layers 1.. in hw["more"]."""
    return hw if i == 0 else hw["more"][i - 1]


def head_context_kv(sh: Shape, hw: dict, feats: torch.Tensor, pos: torch.Tensor):
    """K/V rows a head layer keeps for committed positions: projections of rms(feature) * g_ctx, keys rotated.
    `hw` is that layer's weight dict; `feats` the hidden states of the target layer it taps."""
    hn = rmsnorm(feats, hw["ctx_norm"], sh.rms_eps)
    _, k, v = split_qkv(sh, hn @ hw["wqkv"].T)
    return rope(k, pos, sh.rope_theta), v


def _set_head_rows(sh: Shape, hw: dict, st: "SeqState", rows: torch.Tensor, tap_hidden: Sequence[torch.Tensor]) -> None:
    """Store the tapped features of `rows` and fold them into every head layer's context K/V."""
    for i, f in enumerate(tap_hidden):
        feat = st.feat if i == 0 else st.feat_more[i - 1]
        hK = st.hK if i == 0 else st.hK_more[i - 1]
        hV = st.hV if i == 0 else st.hV_more[i - 1]
        feat[rows] = f
        hK[rows], hV[rows] = head_context_kv(sh, head_layer(hw, i), f, rows)


def _taps_of(hidden: torch.Tensor) -> List[torch.Tensor]:
    """hidden [n,H] (one tap) or [T,n,H] (one slice per head layer) -> list of [n,H]."""
    return [hidden] if hidden.dim() == 2 else [hidden[i] for i in range(hidden.shape[0])]


def prefill(sh: Shape, tw: dict, hw: dict, ctx_embeds: torch.Tensor, cap: int) -> SeqState:
    """Causal forward over the context; fills caches; root = greedy token after the context."""
    P = ctx_embeds.shape[0]
    pos = torch.arange(P)
    mask = torch.tril(torch.ones(P, P, dtype=torch.bool))
    x = ctx_embeds.clone()
    Ks, Vs = [], []
    tapped = {}
    for l, lw in enumerate(tw["layers"]):
        Kc = torch.zeros(cap, sh.n_kv_heads, sh.head_dim)
        Vc = torch.zeros(cap, sh.n_kv_heads, sh.head_dim)
        x = decoder_layer(sh, lw, x, pos, Kc, Vc, pos, mask)
        Ks.append(Kc); Vs.append(Vc)
        if l in sh.taps:
            tapped[l] = x
    logits = rmsnorm(x[-1:], tw["final_norm"], sh.rms_eps) @ tw["lm_head"].T
    root = int(argmax_lowest(logits)[0])
    T = len(sh.taps)
    zkv = lambda: torch.zeros(cap, sh.n_kv_heads, sh.head_dim)
    st = SeqState(P, root, Ks, Vs, zkv(), zkv(), torch.zeros(cap, sh.hidden),
                  hK_more=[zkv() for _ in range(T - 1)], hV_more=[zkv() for _ in range(T - 1)],
                  feat_more=[torch.zeros(cap, sh.hidden) for _ in range(T - 1)])
    _set_head_rows(sh, hw, st, pos, [tapped[t] for t in sh.taps])
    return st


def draft_block(sh: Shape, tw: dict, hw: dict, st: SeqState, B: int) -> torch.Tensor:
    """Algorithm 1 line 1: one pass of the block head.  Returns logits [B,V]; row j (j >= 1) is offset j.

    Slot 0 holds E[root], slots 1..B-1 the mask embedding; every slot attends to all P
    context keys and all B block keys (no in-block mask).
    """
    P = st.P
    X = hw["mask_embed"][None, :].repeat(B, 1)
    X[0] = tw["embed"][st.root]
    pos = torch.arange(P, P + B)
    mask = torch.ones(B, P + B, dtype=torch.bool)
    for i in range(len(sh.taps)):
        # head layer i: context keys/values come from the target layer it taps, block rows from the layer below
        lw = head_layer(hw, i)
        hK = st.hK if i == 0 else st.hK_more[i - 1]
        hV = st.hV if i == 0 else st.hV_more[i - 1]
        hn = rmsnorm(X, lw["ln1"], sh.rms_eps)
        q, k, v = split_qkv(sh, hn @ lw["wqkv"].T)
        q = rope(q, pos, sh.rope_theta)
        k = rope(k, pos, sh.rope_theta)
        K = torch.cat([hK[:P], k], dim=0)
        V = torch.cat([hV[:P], v], dim=0)
        o = attention(q, K, V, mask)
        X = X + o.reshape(B, -1) @ lw["wo"].T
        h2 = rmsnorm(X, lw["ln2"], sh.rms_eps)
        X = X + mlp(sh, h2, lw["wgu"], lw["wd"])
    return rmsnorm(X, hw["final_norm"], sh.rms_eps) @ tw["lm_head"].T


def topk_logprobs(logits: torch.Tensor, k: int):
    """Per offset j = 1..L: the k largest logits (ties to the lowest id) and lp = logit - lse over the full vocabulary.

    logits [B,V] (row 0 ignored) -> ids [L][k] int32, lp [L][k] float32.
    """
    B, V = logits.shape
    L = B - 1
    ids = np.zeros((L, k), dtype=np.int32)
    lp = np.zeros((L, k), dtype=np.float32)
    for j in range(1, B):
        row = logits[j].numpy()
        order = np.lexsort((np.arange(V), -row))[:k]      # by logit descending, then id ascending
        m = np.float32(row.max())
        lse = np.float32(m + np.log(np.sum(np.exp((row - m).astype(np.float32)), dtype=np.float32)))
        ids[j - 1] = order
        lp[j - 1] = (row[order] - lse).astype(np.float32)
    return ids, lp


def verify_tree(sh: Shape, tw: dict, st: SeqState, tree: Tree, row_embeds: Optional[torch.Tensor] = None):
    """Algorithm 1 lines 3-4: the packed ancestor-masked target pass.

    Row i = node i at position P+depth[i]; K/V of node i written to cache row P+i;
    returns (logits [N,V], hidden [N,H]) with hidden = the residual stream after the tapped target layer (the last
    one for the one-layer head: the pre-final-norm stream); [T,N,H] for a head of T layers.
    """
    P, N = st.P, tree.N
    x = tw["embed"][torch.as_tensor(tree.token, dtype=torch.long)].clone() if row_embeds is None else row_embeds.clone()
    pos = torch.as_tensor(P + tree.depth.astype(np.int64))
    rows = torch.arange(P, P + N)
    mask = visibility(tree, P)
    tapped = {}
    for l, lw in enumerate(tw["layers"]):
        x = decoder_layer(sh, lw, x, pos, st.K[l], st.V[l], rows, mask)
        if l in sh.taps:
            tapped[l] = x
    logits = rmsnorm(x, tw["final_norm"], sh.rms_eps) @ tw["lm_head"].T
    if len(sh.taps) == 1:
        return logits, tapped[sh.taps[0]]
    return logits, torch.stack([tapped[t] for t in sh.taps])     # [T,N,H], one slice per head layer


def walk(tree: Tree, argmax: np.ndarray):
    """Algorithm 1 lines 5-12.  Returns (a, path [a+1] node indices with path[0]=0, out tokens [a], new root)."""
    v = 0
    path = [0]
    out: List[int] = []
    while True:
        t = int(argmax[v])
        child = -1
        for c in range(1, tree.n_nodes):
            if int(tree.parent[c]) == v and int(tree.token[c]) == t:
                child = c
                break
        if child < 0:
            return len(out), path, out, t
        out.append(t)
        v = child
        path.append(v)


def commit(sh: Shape, hw: dict, st: SeqState, path: Sequence[int], hidden: torch.Tensor, out: Sequence[int],
           new_root: int) -> None:
    """Keep the accepted path: cache row P+path[d] -> row P+d (ascending d), append features and head K/V, P += a+1."""
    P = st.P
    a = len(path) - 1
    for l in range(len(st.K)):
        for dd in range(1, a + 1):
            st.K[l][P + dd] = st.K[l][P + path[dd]].clone()
            st.V[l][P + dd] = st.V[l][P + path[dd]].clone()
    idx = torch.as_tensor(list(path), dtype=torch.long)
    pos = torch.arange(P, P + a + 1)
    _set_head_rows(sh, hw, st, pos, [h[idx] for h in _taps_of(hidden)])
    st.tokens.extend([st.root] + [int(t) for t in out])
    st.P = P + a + 1
    st.root = int(new_root)


def spec_round(sh: Shape, tw: dict, hw: dict, st: SeqState, B: int, k: int, N: int, tree: Optional[Tree] = None):
    """One full round (Algorithm 1).  With `tree` given, the draft steps are skipped and that tree is verified."""
    info = {}
    if tree is None:
        dl = draft_block(sh, tw, hw, st, B)
        ids, lp = topk_logprobs(dl, k)
        tree = build_tree(st.root, ids, lp, N)
        info.update(draft_logits=dl, ids=ids, lp=lp)
    logits, hidden = verify_tree(sh, tw, st, tree)
    am = argmax_lowest(logits)
    a, path, out, new_root = walk(tree, am)
    top2 = torch.topk(logits, 2, dim=-1).values
    info.update(tree=tree, logits=logits, hidden=hidden, argmax=am, a=a, path=path, out=out, new_root=new_root,
                margins=(top2[:, 0] - top2[:, 1]).numpy())
    commit(sh, hw, st, path, hidden, out, new_root)
    return info


# ----------------------------------------------------------------------------------------------
# sampling mode (Limitations: under sampling the walk draws each token from the verified row of its
# node and descends while the draw is a child; every committed token is a draw from the target)
# ----------------------------------------------------------------------------------------------
# A draw from softmax(logits / T) is taken as argmax_v (logits[v] / T + g[v]) with g[v] i.i.d. standard Gumbel
# (the Gumbel-max identity).  The noise is a fixed field g(seed, position of the token being drawn, v) from a
# counter-based generator (Philox4x32-10), so that the token drawn at a position does not depend on which tree
# row, round or decoding scheme asks for it: tree rounds then commit exactly the tokens that plain ancestral
# sampling with the same field emits (sampled_ar_cachefree), which is what the sampling walk promises.

_PHILOX_M0, _PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
_PHILOX_W0, _PHILOX_W1 = 0x9E3779B9, 0xBB67AE85


def philox4x32(counter, key, rounds: int = 10) -> np.ndarray:
    """Philox4x32 (Salmon et al., SC 2011).  counter: 4 arrays of uint32 (broadcastable), key: 2 uint32.
    Returns uint32 [4, ...]."""
    mask = np.uint64(0xFFFFFFFF)
    c = [np.asarray(x, dtype=np.uint64) & mask for x in counter]
    c = list(np.broadcast_arrays(*c))
    k0, k1 = np.uint64(int(key[0]) & 0xFFFFFFFF), np.uint64(int(key[1]) & 0xFFFFFFFF)
    for _ in range(rounds):
        p0 = np.uint64(_PHILOX_M0) * c[0]
        p1 = np.uint64(_PHILOX_M1) * c[2]
        hi0, lo0 = p0 >> np.uint64(32), p0 & mask
        hi1, lo1 = p1 >> np.uint64(32), p1 & mask
        c = [(hi1 ^ c[1] ^ k0) & mask, lo1, (hi0 ^ c[3] ^ k1) & mask, lo0]
        k0 = (k0 + np.uint64(_PHILOX_W0)) & mask
        k1 = (k1 + np.uint64(_PHILOX_W1)) & mask
    return np.stack(c).astype(np.uint32)


def uniform_field(seed: int, position: int, V: int) -> np.ndarray:
    """u[v] in (0,1), fp32 exact: vocabulary ids 4b..4b+3 take the four words of Philox(counter = (b, position, 0, 0),
    key = (seed low, seed high)); u = ((word >> 9) + 0.5) * 2^-23."""
    nb = (V + 3) // 4
    words = philox4x32((np.arange(nb, dtype=np.uint64), np.uint64(position & 0xFFFFFFFF), np.uint64(0), np.uint64(0)),
                       (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))
    flat = words.T.reshape(-1)[:V]                                   # id 4b+j <- word j of block b
    return ((flat >> np.uint32(9)).astype(np.float32) + np.float32(0.5)) * np.float32(2.0 ** -23)


def gumbel_field(seed: int, position: int, V: int) -> np.ndarray:
    """Standard Gumbel noise g = -log(-log u) in fp32."""
    u = uniform_field(seed, position, V)
    return (-np.log(-np.log(u))).astype(np.float32)


def perturbed_rows(logits: torch.Tensor, positions: Sequence[int], seed: int, inv_temperature: float = 1.0) -> np.ndarray:
    """y[i][v] = logits[i][v] * inv_temperature + g(seed, positions[i], v), fp32.  positions[i] is the position of
    the token that row i predicts (its own position + 1)."""
    L = logits.numpy().astype(np.float32)
    out = np.empty_like(L)
    for i, pos in enumerate(positions):
        out[i] = L[i] * np.float32(inv_temperature) + gumbel_field(seed, int(pos), L.shape[1])
    return out


def sample_rows(logits: torch.Tensor, positions: Sequence[int], seed: int, inv_temperature: float = 1.0):
    """One draw per row from softmax(logits * inv_temperature): arg-max of the perturbed row, ties to the lowest id.
    Returns (ids int32 [n], margins [n] = gap between the two largest perturbed values)."""
    y = torch.from_numpy(perturbed_rows(logits, positions, seed, inv_temperature))
    top2 = torch.topk(y, 2, dim=-1).values
    return argmax_lowest(y), (top2[:, 0] - top2[:, 1]).numpy()


def sampled_ar_cachefree(sh: Shape, tw: dict, ctx_embeds: torch.Tensor, first: int, n_new: int, seed: int):
    """Plain ancestral sampling at temperature 1, one full causal forward per token, no cache: after the context and
    the given first token (the pending root), token number k is drawn from the target's row with the noise field of
    its own position.  Returns the n_new tokens after `first`."""
    x = torch.cat([ctx_embeds, tw["embed"][first][None, :]], dim=0)
    toks = []
    for _ in range(n_new):
        logits, _ = full_causal_forward(sh, tw, x)
        t = int(sample_rows(logits[-1:], [x.shape[0]], seed)[0][0])
        toks.append(t)
        x = torch.cat([x, tw["embed"][t][None, :]], dim=0)
    return toks


def spec_round_sampled(sh: Shape, tw: dict, hw: dict, st: SeqState, B: int, k: int, N: int, seed: int,
                       tree: Optional[Tree] = None):
    """One round in sampling mode: as spec_round, but every row's decision is a draw from its verified row."""
    info = {}
    if tree is None:
        dl = draft_block(sh, tw, hw, st, B)
        ids, lp = topk_logprobs(dl, k)
        tree = build_tree(st.root, ids, lp, N)
        info.update(draft_logits=dl, ids=ids, lp=lp)
    logits, hidden = verify_tree(sh, tw, st, tree)
    positions = [st.P + int(d) + 1 for d in tree.depth]
    draws, margins = sample_rows(logits, positions, seed)
    a, path, out, new_root = walk(tree, draws)
    info.update(tree=tree, logits=logits, hidden=hidden, argmax=draws, a=a, path=path, out=out, new_root=new_root,
                margins=margins)
    commit(sh, hw, st, path, hidden, out, new_root)
    return info


# ----------------------------------------------------------------------------------------------
# acceptance statistics (Eq. 1, Eq. 2)
# ----------------------------------------------------------------------------------------------

def root_entropy(logits_row: torch.Tensor) -> float:
    """Section 4: the target's next-token entropy at the round root, H = -sum_v p_v log p_v in nats, p = softmax of
    the root row's logits; computed as lse - sum_v p_v * logit_v in float64."""
    x = logits_row.double()
    lse = torch.logsumexp(x, dim=-1)
    p = torch.exp(x - lse)
    return float(lse - (p * x).sum())


def expected_accept(p_m: float, L: int) -> float:
    """Eq. 2: E[a | p_m] = sum_{l=1..L} p_m^l."""
    return float(sum(p_m ** l for l in range(1, L + 1)))


def mean_accept_tokens(accept_lengths: Sequence[int]) -> float:
    """Eq. 1: tau = E[a] + 1."""
    return float(np.mean(np.asarray(accept_lengths, dtype=np.float64)) + 1.0)
