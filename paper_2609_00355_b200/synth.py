"""Seeded synthetic inputs for one GLANCE speculative round.

This module only *draws* inputs (weights, contexts, top-k marginals, random trees).
It holds none of the method's arithmetic: no model forward, no tree scoring, no
masks, no acceptance.  Both the CPU oracle's tests and the CUDA library's callers
obtain their inputs here so that the two sides see the same bits.

Recipe (all tensors bf16 unless noted):
  * weights: every matrix N(0, 0.02) drawn with one seeded ``torch.Generator`` in a
    fixed order (embed, lm_head, then per layer wqkv, wo, wgu, wd, then the head's
    mask_embed, wqkv, wo, wgu, wd); every RMSNorm gain is 1.0.
  * context: ``n_img`` "image" rows of N(0, 1) embeddings placed first, followed by
    ``n_txt`` uniform random token ids (the paper's regime: image tokens outnumber
    text tokens and vision enters as a token prefix).
  * controlled-match marginals: every depth has the same top-k distribution
    q[0] = p_m, q[r] = (1 - p_m) 2^-r; the true continuation token is placed at
    rank 0 with probability p_m and is otherwise absent from the candidates.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class RoundConfig:
    name: str
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    n_img: int
    n_txt: int
    block_B: int
    topk: int
    tree_N: int
    p_m: float
    rounds: int
    batch: int = 1
    page_size: int = 64
    rms_eps: float = 1e-6
    rope_theta: float = 1e6
    # () = one head layer fed by the last target layer; otherwise head layer i reads the hidden states after
    # target layer head_taps[i] (0-based), one tap per head layer (Section 3.2: five layers, five kept target layers)
    head_taps: tuple = ()

    @property
    def head_layers(self) -> int:
        return max(1, len(self.head_taps))

    @property
    def L(self) -> int:
        return self.block_B - 1

    @property
    def ctx(self) -> int:
        return self.n_img + self.n_txt

    @property
    def G(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def replace(self, **kw) -> "RoundConfig":
        return dataclasses.replace(self, **kw)


CONFIGS: Dict[str, RoundConfig] = {
    "tiny": RoundConfig("tiny", 2, 256, 4, 2, 64, 704, 1024, 256, 64, 4, 2, 8, 0.7, 16),
    "small": RoundConfig("small", 8, 1024, 16, 4, 64, 2816, 32000, 576, 128, 8, 4, 32, 0.6, 64),
    "7b": RoundConfig("7b", 28, 3584, 28, 4, 128, 18944, 152064, 1280, 256, 16, 8, 64, 0.8, 128),
    "long": RoundConfig("long", 28, 3584, 28, 4, 128, 18944, 152064, 8192, 512, 16, 8, 128, 0.5, 64),
    "batch8": RoundConfig("batch8", 28, 3584, 28, 4, 128, 18944, 152064, 3072, 1024, 16, 8, 64, 0.65, 128, batch=8),
}


def _normal_bf16(shape, std, gen, device):
    # drawn in fp32 on `device`, scaled, rounded to bf16 (round-to-nearest-even)
    return (torch.randn(shape, generator=gen, device=device, dtype=torch.float32) * std).to(torch.bfloat16)


def make_weights(cfg: RoundConfig, device="cpu", seed: int = 0):
    """Random-init target decoder + one-layer draft head.  Returns (target, head) dicts.

    target: embed [V,H], lm_head [V,H], final_norm [H], layers: list of dicts with
            ln1 [H], wqkv [(Hq+2Hkv)d, H], wo [H, Hq d], ln2 [H], wgu [2F, H], wd [H, F]
    head:   mask_embed [H], ctx_norm [H], ln1, wqkv, wo, ln2, wgu, wd, final_norm
            (embed and lm_head are shared with the target); with cfg.head_taps of T > 1 entries also
            more: list of T-1 dicts {ctx_norm, ln1, wqkv, wo, ln2, wgu, wd} for head layers 1..T-1
    """
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    H, d, F, V = cfg.hidden, cfg.head_dim, cfg.ffn, cfg.vocab
    qkv_out = (cfg.n_q_heads + 2 * cfg.n_kv_heads) * d
    ones = lambda: torch.ones(H, dtype=torch.bfloat16, device=device)
    std = 0.02
    target = {
        "embed": _normal_bf16((V, H), std, gen, device),
        "lm_head": _normal_bf16((V, H), std, gen, device),
        "final_norm": ones(),
        "layers": [],
    }
    for _ in range(cfg.n_layers):
        target["layers"].append({
            "ln1": ones(),
            "wqkv": _normal_bf16((qkv_out, H), std, gen, device),
            "wo": _normal_bf16((H, cfg.n_q_heads * d), std, gen, device),
            "ln2": ones(),
            "wgu": _normal_bf16((2 * F, H), std, gen, device),
            "wd": _normal_bf16((H, F), std, gen, device),
        })
    head = {
        "mask_embed": _normal_bf16((H,), std, gen, device),
        "ctx_norm": ones(),
        "ln1": ones(),
        "wqkv": _normal_bf16((qkv_out, H), std, gen, device),
        "wo": _normal_bf16((H, cfg.n_q_heads * d), std, gen, device),
        "ln2": ones(),
        "wgu": _normal_bf16((2 * F, H), std, gen, device),
        "wd": _normal_bf16((H, F), std, gen, device),
        "final_norm": ones(),
    }
    # head layers 1.. (drawn after everything else, so a one-layer head keeps its bits)
    more = []
    for _ in range(cfg.head_layers - 1):
        more.append({
            "ctx_norm": ones(),
            "ln1": ones(),
            "wqkv": _normal_bf16((qkv_out, H), std, gen, device),
            "wo": _normal_bf16((H, cfg.n_q_heads * d), std, gen, device),
            "ln2": ones(),
            "wgu": _normal_bf16((2 * F, H), std, gen, device),
            "wd": _normal_bf16((H, F), std, gen, device),
        })
    if more:
        head["more"] = more
    return target, head


def make_context(cfg: RoundConfig, device="cpu", seed: int = 1, n_img: Optional[int] = None,
                 n_txt: Optional[int] = None):
    """Returns (image_embeds [n_img,H] bf16, text_ids [n_txt] int32)."""
    n_img = cfg.n_img if n_img is None else n_img
    n_txt = cfg.n_txt if n_txt is None else n_txt
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    img = torch.randn((n_img, cfg.hidden), generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)
    ids = torch.randint(0, cfg.vocab, (n_txt,), generator=gen, device=device, dtype=torch.int64).to(torch.int32)
    return img, ids


def batch_context_lengths(cfg: RoundConfig, lo: int = 1024, hi: int = 4096, seed: int = 2) -> List[int]:
    """Per-sequence context lengths of the small-batch serving config (uniform in [lo, hi])."""
    rng = np.random.default_rng(seed)
    return [int(x) for x in rng.integers(lo, hi + 1, size=cfg.batch)]


def batch_match_probs(cfg: RoundConfig, lo: float = 0.4, hi: float = 0.9, seed: int = 4) -> List[float]:
    rng = np.random.default_rng(seed)
    return [float(x) for x in rng.uniform(lo, hi, size=cfg.batch)]


def controlled_marginals(p_m: float, k: int, L: int) -> np.ndarray:
    """Log-probabilities lp[L][k] (fp32) of the controlled-match marginals; same row at every depth."""
    q = [p_m] + [(1.0 - p_m) * 2.0 ** (-r) for r in range(1, k)]
    row = np.array([math.log(x) for x in q], dtype=np.float32)
    return np.tile(row[None, :], (L, 1))


def controlled_candidates(Y: List[int], p_m: float, k: int, L: int, vocab: int,
                          rng: np.random.Generator) -> np.ndarray:
    """Candidate ids[L][k] (int32) for one round.

    Y[j] is the target's true greedy token at depth j+1.  With probability p_m
    (independently per depth) it sits at rank 0; otherwise it is absent from that
    depth's candidates.  All other candidates are distinct random ids != Y[j].
    """
    ids = np.zeros((L, k), dtype=np.int32)
    for j in range(L):
        y = int(Y[j])
        hit = rng.random() < p_m
        others: List[int] = []
        while len(others) < k:
            c = int(rng.integers(0, vocab))
            if c != y and c not in others:
                others.append(c)
        row = others
        if hit:
            row = [y] + others[: k - 1]
        ids[j] = np.array(row, dtype=np.int32)
    return ids


def calibrated_candidates(Y: List[int], p_m: float, k: int, L: int, vocab: int,
                          rng: np.random.Generator) -> np.ndarray:
    """Candidate ids[L][k] whose ranks are calibrated to the controlled marginals: the true token Y[j] sits at rank
    r with probability q[r] (q[0] = p_m, q[r] = (1 - p_m) 2^-r) and is absent with the remaining mass, so that
    sibling branches of a tree can be hit (budget sweeps); other candidates are distinct random ids != Y[j]."""
    q = [p_m] + [(1.0 - p_m) * 2.0 ** (-r) for r in range(1, k)]
    ids = np.zeros((L, k), dtype=np.int32)
    for j in range(L):
        y = int(Y[j])
        u, r_hit, acc = rng.random(), -1, 0.0
        for r in range(k):
            acc += q[r]
            if u < acc:
                r_hit = r
                break
        others: List[int] = []
        while len(others) < k:
            c = int(rng.integers(0, vocab))
            if c != y and c not in others:
                others.append(c)
        if r_hit >= 0:
            others[r_hit] = y
        ids[j] = np.array(others, dtype=np.int32)
    return ids


def random_topk(L: int, k: int, vocab: int, rng: np.random.Generator, ties: bool = False):
    """Random per-depth candidates: distinct ids and non-increasing fp32 log-probs (for tree-builder tests)."""
    ids = np.zeros((L, k), dtype=np.int32)
    lp = np.zeros((L, k), dtype=np.float32)
    for j in range(L):
        ids[j] = rng.choice(vocab, size=k, replace=False).astype(np.int32)
        if ties:
            vals = -rng.integers(1, 4, size=k).astype(np.float32) * np.float32(0.25)
        else:
            vals = np.log(rng.dirichlet(np.ones(k) * 0.7) * 0.9 + 1e-9).astype(np.float32)
        lp[j] = np.sort(vals)[::-1]
    return ids, lp


def random_tree(n_nodes: int, L: int, vocab: int, rng: np.random.Generator, tokens_for=None):
    """A random prefix-closed candidate tree in topological order (parent index < child index).

    Returns (token, parent, depth) int32 arrays of length n_nodes; node 0 is the root
    (token filled by the caller).  Sibling tokens are distinct.  ``tokens_for(parent, depth)``
    may supply a preferred token for the first child of a node (used to plant the true
    continuation so that some paths are accepted).
    """
    token = np.zeros(n_nodes, dtype=np.int32)
    parent = np.full(n_nodes, -1, dtype=np.int32)
    depth = np.zeros(n_nodes, dtype=np.int32)
    children: Dict[int, List[int]] = {0: []}
    for i in range(1, n_nodes):
        cands = [p for p in range(i) if depth[p] < L]
        p = int(cands[int(rng.integers(0, len(cands)))])
        parent[i] = p
        depth[i] = depth[p] + 1
        used = {int(token[c]) for c in children[p]}
        t = None
        if tokens_for is not None and not children[p]:
            t = tokens_for(p, int(depth[i]))
        while t is None or t in used:
            t = int(rng.integers(0, vocab))
        token[i] = t
        children[p].append(i)
        children[i] = []
    return token, parent, depth
