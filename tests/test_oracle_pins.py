"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test is chosen so that a plausible mistake in the oracle (dropped term, wrong sign or
index, transposed operand, wrong mask bit) fails it.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import glance_oracle as O
from paper_2609_00355_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ Eq. 1 / Eq. 2: printed values

def _golden_rows():
    rows = []
    with open(os.path.join(GOLDEN, "eq2_printed_values.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            kind, arg, L, val, dec = line.split()
            rows.append((kind, float(arg), int(L), float(val), int(dec)))
    return rows


def test_eq2_printed_values():
    """Eq. 2 / Lemma 1: the closed form reproduces every number the paper prints for it."""
    sig = lambda z: 1.0 / (1.0 + math.exp(-z))
    seen = set()
    for kind, arg, L, val, dec in _golden_rows():
        half = 0.5 * 10.0 ** (-dec) + 1e-12
        seen.add(kind)
        if kind == "trunc_err":
            p = arg
            trunc = O.expected_accept(p, L)
            untr = p / (1.0 - p)
            assert abs((untr - trunc) / untr - val) <= half
            assert abs(p ** L - val) <= half
        elif kind == "sup_mean":
            assert abs(O.expected_accept(sig(arg), L) - val) <= half
        elif kind == "geo_cap":
            p = sig(arg)
            assert abs(p / (1 - p) - val) <= half and abs(math.exp(arg) - val) <= half
        elif kind == "rel_gap_bound":
            for p in np.linspace(0.05, arg, 16):
                untr = p / (1 - p)
                assert (untr - O.expected_accept(float(p), L)) / untr < val
    assert seen == {"trunc_err", "sup_mean", "geo_cap", "rel_gap_bound"}


def test_eq2_closed_form_and_eq1():
    for p in (0.3, 0.5, 0.8, 0.9):
        for L in (1, 3, 7, 15):
            assert abs(O.expected_accept(p, L) - p * (1 - p ** L) / (1 - p)) < 1e-12
    assert O.mean_accept_tokens([0, 0, 0]) == 1.0          # autoregressive decoding has tau = 1
    assert O.mean_accept_tokens([2, 4]) == 4.0


# ------------------------------------------------------------------ model pieces

def test_rmsnorm_closed_form():
    x = torch.tensor([[3.0, -4.0, 0.0, 0.0]])
    g = torch.tensor([1.0, 2.0, 1.0, 1.0])
    y = O.rmsnorm(x, g, 0.0)
    rms = math.sqrt(25.0 / 4.0)
    assert torch.allclose(y, torch.tensor([[3.0 / rms, -8.0 / rms, 0.0, 0.0]]), atol=1e-6)
    c = torch.full((2, 8), 5.0)
    assert torch.allclose(O.rmsnorm(c, torch.ones(8), 0.0), torch.ones(2, 8), atol=1e-6)


def test_rope_pairs_and_relative_position():
    # d = 2: one pair (0, 1), frequency theta^0 = 1: (1, 0) at position p -> (cos p, sin p)
    x = torch.tensor([[[1.0, 0.0]]])
    y = O.rope(x, torch.tensor([2]), 1e6)
    assert torch.allclose(y, torch.tensor([[[math.cos(2.0), math.sin(2.0)]]]), atol=1e-6)
    # d = 4: pairs are (0, 2) and (1, 3); second pair rotates by p * theta^(-1/2)
    x = torch.tensor([[[0.0, 1.0, 0.0, 0.0]]])
    y = O.rope(x, torch.tensor([3]), 100.0)
    assert torch.allclose(y, torch.tensor([[[0.0, math.cos(0.3), 0.0, math.sin(0.3)]]]), atol=1e-6)
    # position 0 is the identity; rotation preserves norms; scores depend on position differences only
    g = torch.Generator().manual_seed(0)
    q = torch.randn(1, 3, 16, generator=g)
    k = torch.randn(1, 3, 16, generator=g)
    assert torch.allclose(O.rope(q, torch.tensor([0]), 1e4), q)
    assert torch.allclose(O.rope(q, torch.tensor([77]), 1e4).norm(dim=-1), q.norm(dim=-1), atol=1e-5)
    s1 = (O.rope(q, torch.tensor([40]), 1e4) * O.rope(k, torch.tensor([33]), 1e4)).sum(-1)
    s2 = (O.rope(q, torch.tensor([12]), 1e4) * O.rope(k, torch.tensor([5]), 1e4)).sum(-1)
    s3 = (O.rope(q, torch.tensor([12]), 1e4) * O.rope(k, torch.tensor([6]), 1e4)).sum(-1)
    assert torch.allclose(s1, s2, atol=1e-4)
    assert not torch.allclose(s1, s3, atol=1e-3)


def test_attention_matches_library_sdpa():
    g = torch.Generator().manual_seed(1)
    n, m, Hq, Hkv, d = 9, 23, 6, 2, 16
    q = torch.randn(n, Hq, d, generator=g)
    K = torch.randn(m, Hkv, d, generator=g)
    V = torch.randn(m, Hkv, d, generator=g)
    mask = torch.rand(n, m, generator=g) < 0.6
    mask[:, 0] = True
    got = O.attention(q, K, V, mask)
    Kr = K.repeat_interleave(Hq // Hkv, dim=1)
    Vr = V.repeat_interleave(Hq // Hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(
        q.transpose(0, 1)[None], Kr.transpose(0, 1)[None], Vr.transpose(0, 1)[None], attn_mask=mask[None, None])
    assert torch.allclose(got, ref[0].transpose(0, 1), atol=1e-5)


def test_topk_logprobs_matches_library_and_breaks_ties_low():
    g = torch.Generator().manual_seed(2)
    logits = torch.randn(5, 300, generator=g) * 3
    logits[2, 17] = logits[2, 250] = logits[2].max() + 1.0       # exact tie for rank 0 of offset 2
    ids, lp = O.topk_logprobs(logits, 4)
    assert ids.shape == (4, 4)
    for j in range(1, 5):
        tv, ti = torch.topk(logits[j], 4)
        lse = torch.logsumexp(logits[j].double(), dim=-1)
        assert np.allclose(lp[j - 1], (tv.double() - lse).numpy(), atol=1e-5)
        if j != 2:
            assert list(ids[j - 1]) == ti.tolist()
        assert np.all(np.diff(lp[j - 1]) <= 0) and np.all(lp[j - 1] <= 0)
    assert list(ids[1][:2]) == [17, 250]
    # probabilities of the full vocabulary sum to one
    ids_all, lp_all = O.topk_logprobs(logits[:2], 300)
    assert abs(np.exp(lp_all[0].astype(np.float64)).sum() - 1.0) < 1e-4


def test_argmax_lowest_id_on_ties():
    x = torch.tensor([[1.0, 5.0, 5.0, 2.0], [7.0, 1.0, 7.0, 7.0]])
    assert list(O.argmax_lowest(x)) == [1, 0]


# ------------------------------------------------------------------ candidate tree

def _assert_tree_equal(a: O.Tree, b: O.Tree):
    assert a.n_nodes == b.n_nodes
    for f in ("token", "parent", "depth", "rank"):
        assert np.array_equal(getattr(a, f), getattr(b, f)), f
    assert np.array_equal(a.score.view(np.uint32), b.score.view(np.uint32))
    assert np.array_equal(a.anc, b.anc)


@pytest.mark.parametrize("L,k,N", [(3, 2, 8), (3, 2, 16), (4, 3, 32), (7, 4, 32), (5, 8, 64), (2, 2, 64)])
@pytest.mark.parametrize("ties", [False, True])
def test_best_first_equals_bruteforce_sort(L, k, N, ties):
    """Algorithm 1 line 2: best-first search returns exactly the sorted top N-1 prefixes."""
    rng = np.random.default_rng(100 * L + k + (7 if ties else 0))
    if k ** L > 40000:
        pytest.skip("enumeration too large")
    for _ in range(3):
        ids, lp = synth.random_topk(L, k, 5000, rng, ties=ties)
        _assert_tree_equal(O.build_tree(11, ids, lp, N), O.build_tree_bruteforce(11, ids, lp, N))


def test_best_first_on_controlled_marginals_with_exact_score_ties():
    # identical marginals at every depth: commuted sums tie exactly, the path key decides
    lp = synth.controlled_marginals(0.8, 4, 6)
    ids = np.arange(24, dtype=np.int32).reshape(6, 4)
    bf, bb = O.build_tree(3, ids, lp, 64), O.build_tree_bruteforce(3, ids, lp, 64)
    _assert_tree_equal(bf, bb)
    sc = bf.score[1:bf.n_nodes]
    assert len(np.unique(sc)) < len(sc)


def test_tree_invariants():
    """Section 3.3: the kept set is prefix-closed; no prefix scores below its extensions."""
    rng = np.random.default_rng(5)
    ids, lp = synth.random_topk(15, 8, 152064, rng)
    t = O.build_tree(9, ids, lp, 64)
    assert t.n_nodes == 64 and t.parent[0] == -1 and t.depth[0] == 0
    for i in range(1, t.n_nodes):
        p = t.parent[i]
        assert 0 <= p < i and t.depth[i] == t.depth[p] + 1
        assert t.score[i] <= t.score[p]
        assert t.token[i] == ids[t.depth[i] - 1][t.rank[i]]
        assert np.float32(t.score[p] + lp[t.depth[i] - 1][t.rank[i]]) == t.score[i]
    assert np.all(np.diff(t.score[1:t.n_nodes]) <= 0)
    # fewer candidates than rows: n_nodes reported, padding rows see only themselves
    ids2, lp2 = synth.random_topk(2, 2, 100, rng)
    t2 = O.build_tree(1, ids2, lp2, 16)
    assert t2.n_nodes == 1 + 2 + 4
    for i in range(t2.n_nodes, 16):
        assert t2.parent[i] == -1 and int(t2.anc[i, 0]) == 1 << i


EX_PARENT = [-1, 0, 0, 1, 1, 2, 3, 4]
EX_DEPTH = [0, 1, 1, 2, 2, 2, 3, 3]
EX_TOKEN = [7, 11, 12, 21, 22, 23, 31, 32]


def test_ancestor_mask_hand_example():
    # hand-derived: node 6 -> ancestors 3, 1, 0 -> bits {0,1,3,6} = 0x4B, node 7 -> {0,1,4,7} = 0x93
    t = O.tree_from_arrays(EX_TOKEN, EX_PARENT, EX_DEPTH)
    assert [int(x) for x in t.anc[:, 0]] == [0x01, 0x03, 0x05, 0x0B, 0x13, 0x25, 0x4B, 0x93]
    big = O.chain_tree(1, list(range(2, 72)), 128)             # second mask word
    assert int(big.anc[70, 1]) == (1 << 7) - 1 and int(big.anc[70, 0]) == (1 << 64) - 1
    assert int(big.anc[100, 0]) == 0 and int(big.anc[100, 1]) == 1 << 36


def test_walk_hand_examples():
    """Algorithm 1 lines 5-12 on a hand-made tree."""
    t = O.tree_from_arrays(EX_TOKEN, EX_PARENT, EX_DEPTH)
    am = np.array([11, 22, 0, 0, 99, 0, 0, 0])
    assert O.walk(t, am) == (2, [0, 1, 4], [11, 22], 99)
    am = np.array([12, 0, 23, 0, 0, 5, 0, 0])                  # node 5 is a leaf: stop there
    assert O.walk(t, am) == (2, [0, 2, 5], [12, 23], 5)
    am = np.array([13, 0, 0, 0, 0, 0, 0, 0])
    assert O.walk(t, am) == (0, [0], [], 13)
    am = np.array([11, 21, 0, 31, 0, 0, 44, 0])                # full depth
    assert O.walk(t, am) == (3, [0, 1, 3, 6], [11, 21, 31], 44)
    # a padding row can never be entered even if its token matches
    tp = O.tree_from_arrays(EX_TOKEN[:3], EX_PARENT[:3], EX_DEPTH[:3], N=8)
    assert O.walk(tp, np.array([0, 0, 0, 0, 0, 0, 0, 0])) == (0, [0], [], 0)


def test_masks_chain_is_causal_and_star_sees_root_and_self():
    P = 5
    ch = O.chain_tree(1, [2, 3, 4, 5], 5)
    m = O.visibility(ch, P)
    assert torch.equal(m[:, :P], torch.ones(5, P, dtype=torch.bool))
    assert torch.equal(m[:, P:], torch.tril(torch.ones(5, 5, dtype=torch.bool)))
    star = O.tree_from_arrays([1, 2, 3, 4], [-1, 0, 0, 0], [0, 1, 1, 1])
    ms = O.visibility(star, 0)
    expect = torch.eye(4, dtype=torch.bool)
    expect[:, 0] = True
    assert torch.equal(ms, expect)


# ------------------------------------------------------------------ the round on the tiny config

class Tiny:
    pass


@pytest.fixture(scope="module")
def tiny():
    torch.manual_seed(0)
    cfg = synth.CONFIGS["tiny"]
    tw_b, hw_b = synth.make_weights(cfg)
    img, ids = synth.make_context(cfg)
    t = Tiny()
    t.cfg, t.sh = cfg, O.Shape.of(cfg)
    t.tw, t.hw = O.widen(tw_b), O.widen(hw_b)
    t.ctx = O.context_embeddings(t.tw, img, ids.numpy())
    t.n_new = 40
    t.Y, t.margins = O.greedy_ar_cachefree(t.sh, t.tw, t.ctx, t.n_new)
    t.cap = cfg.ctx + t.n_new + cfg.tree_N + 64
    return t


def _fresh(t):
    return O.prefill(t.sh, t.tw, t.hw, t.ctx, t.cap)


def test_prefill_root_is_first_greedy_token(tiny):
    st = _fresh(tiny)
    assert st.P == tiny.cfg.ctx and st.root == tiny.Y[0]
    print("smallest top-2 margin met by plain greedy decoding:", min(tiny.margins))


def test_verify_rows_equal_plain_chain(tiny):
    """Definition 1: the row of node y_1:d is p(. | x o b o y_1:d), for every node of small trees."""
    rng = np.random.default_rng(3)
    st = _fresh(tiny)
    for n_nodes in (8, 5):
        tok, par, dep = synth.random_tree(n_nodes, tiny.cfg.L, tiny.cfg.vocab, rng)
        tok[0] = st.root
        tree = O.tree_from_arrays(tok, par, dep, N=8)
        logits, hidden = O.verify_tree(tiny.sh, tiny.tw, st, tree)
        scale = float(logits.abs().max())
        for s, i in O.tree_paths(tree).items():
            ref_l, ref_h = O.chain_row(tiny.sh, tiny.tw, tiny.ctx, st.root, s)
            assert float((logits[i] - ref_l).abs().max()) <= 1e-4 * scale
            assert float((hidden[i] - ref_h).abs().max()) <= 1e-4 * float(hidden.abs().max())
        ref_l, _ = O.chain_row(tiny.sh, tiny.tw, tiny.ctx, st.root, ())
        assert float((logits[0] - ref_l).abs().max()) <= 1e-4 * scale


def test_mask_errors_are_visible_in_attention():
    """A wrong mask bit must change the output by O(1): one-hot values, strongly separated keys."""
    n = 6
    K = torch.eye(n)[:, None, :] * 30.0
    V = torch.eye(n)[:, None, :]
    q = torch.ones(n, 1, n)
    tree = O.tree_from_arrays([0] * n, [-1, 0, 0, 1, 1, 2], [0, 1, 1, 2, 2, 2])
    out = O.attention(q, K, V, O.visibility(tree, 0))[:, 0, :]
    for i in range(n):
        vis = [(int(tree.anc[i, 0]) >> j) & 1 for j in range(n)]
        expect = torch.tensor(vis, dtype=torch.float32) / sum(vis)
        assert torch.allclose(out[i], expect, atol=1e-6)


def test_chain_tree_verify_equals_causal_chunk(tiny):
    st = _fresh(tiny)
    chain = O.chain_tree(st.root, tiny.Y[1:8], 8)
    logits, hidden = O.verify_tree(tiny.sh, tiny.tw, st, chain)
    x = torch.cat([tiny.ctx, tiny.tw["embed"][torch.tensor(tiny.Y[:8])]], dim=0)
    ref_l, ref_h = O.full_causal_forward(tiny.sh, tiny.tw, x)
    assert float((logits - ref_l[-8:]).abs().max()) <= 1e-4 * float(ref_l.abs().max())
    assert float((hidden - ref_h[-8:]).abs().max()) <= 1e-4 * float(ref_h.abs().max())
    # and the whole chain is accepted: a = 7 = min(L-limit of the chain, matches)
    a, path, out, new_root = O.walk(chain, O.argmax_lowest(logits))
    assert (a, path, out, new_root) == (7, list(range(8)), tiny.Y[1:8], tiny.Y[8])


def _run_rounds(t, tree_fn, n_rounds):
    st = _fresh(t)
    accepts = []
    for _ in range(n_rounds):
        done = len(st.tokens)
        Yrest = t.Y[done + 1:]
        tree = tree_fn(st, Yrest)
        if len(Yrest) < t.cfg.L + 2:
            break
        info = O.spec_round(t.sh, t.tw, t.hw, st, t.cfg.block_B, t.cfg.topk, t.cfg.tree_N, tree=tree)
        assert info["a"] == O.accepted_length_bruteforce(info["tree"], Yrest)     # Definition 1
        accepts.append(info["a"])
    emitted = st.tokens + [st.root]
    assert emitted == t.Y[:len(emitted)]                                         # Theorem 1
    return st, accepts


def test_lossless_with_drafted_best_first_trees(tiny):
    st, acc = _run_rounds(tiny, lambda st, Y: None, 8)
    assert len(acc) == 8


def test_lossless_with_random_trees_planted_continuation(tiny):
    rng = np.random.default_rng(11)

    def tree_fn(st, Y):
        def pref(parent, depth):
            # plant the true continuation along first children with probability 0.7
            return int(Y[depth - 1]) if rng.random() < 0.7 and depth - 1 < len(Y) else None
        tok, par, dep = synth.random_tree(8, tiny.cfg.L, tiny.cfg.vocab, rng, tokens_for=pref)
        tok[0] = st.root
        return O.tree_from_arrays(tok, par, dep, N=8)

    st, acc = _run_rounds(tiny, tree_fn, 10)
    assert max(acc) >= 1 and min(acc) == 0 or len(set(acc)) > 1


def test_lossless_with_garbage_trees_and_chain_and_single_node(tiny):
    rng = np.random.default_rng(12)

    def garbage(st, Y):
        tok, par, dep = synth.random_tree(8, tiny.cfg.L, tiny.cfg.vocab, rng)
        tok[0] = st.root
        return O.tree_from_arrays(tok, par, dep, N=8)

    _run_rounds(tiny, garbage, 5)
    st, acc = _run_rounds(tiny, lambda st, Y: O.chain_tree(st.root, Y[:3], 8), 6)
    assert acc == [3] * len(acc)                      # a true chain of depth L is accepted whole
    st, acc = _run_rounds(tiny, lambda st, Y: O.chain_tree(st.root, [], 1), 6)
    assert acc == [0] * len(acc) and O.mean_accept_tokens(acc) == 1.0    # N = 1 is plain AR, tau = 1


def test_kv_state_after_rounds_equals_fresh_prefill(tiny):
    rng = np.random.default_rng(13)

    def tree_fn(st, Y):
        def pref(parent, depth):
            return int(Y[depth - 1]) if rng.random() < 0.8 else None
        tok, par, dep = synth.random_tree(8, tiny.cfg.L, tiny.cfg.vocab, rng, tokens_for=pref)
        tok[0] = st.root
        return O.tree_from_arrays(tok, par, dep, N=8)

    st, acc = _run_rounds(tiny, tree_fn, 6)
    assert sum(acc) > 0
    x = torch.cat([tiny.ctx, tiny.tw["embed"][torch.tensor(st.tokens)]], dim=0)
    ref = O.prefill(tiny.sh, tiny.tw, tiny.hw, x, tiny.cap)
    assert ref.P == st.P and ref.root == st.root
    for l in range(tiny.sh.n_layers):
        assert float((ref.K[l][:st.P] - st.K[l][:st.P]).abs().max()) < 1e-4
        assert float((ref.V[l][:st.P] - st.V[l][:st.P]).abs().max()) < 1e-4
    assert float((ref.hK[:st.P] - st.hK[:st.P]).abs().max()) < 1e-4
    assert float((ref.hV[:st.P] - st.hV[:st.P]).abs().max()) < 1e-4
    assert float((ref.feat[:st.P] - st.feat[:st.P]).abs().max()) < 1e-4 * float(ref.feat.abs().max())


def test_commit_moves_rows_in_ascending_order_hazard_case(tiny):
    """Path (0,2,5): cache row P+2 is read by step 1 and overwritten by step 2."""
    st = _fresh(tiny)
    P = st.P
    for l in range(tiny.sh.n_layers):
        for i in range(8):
            st.K[l][P + i] = float(100 * l + i)
            st.V[l][P + i] = float(-100 * l - i)
    hidden = torch.arange(8, dtype=torch.float32)[:, None].repeat(1, tiny.sh.hidden)
    O.commit(tiny.sh, tiny.hw, st, [0, 2, 5], hidden, [12, 23], 5)
    assert st.P == P + 3 and st.root == 5
    for l in range(tiny.sh.n_layers):
        assert [float(st.K[l][P + i, 0, 0]) for i in range(3)] == [100 * l + 0, 100 * l + 2, 100 * l + 5]
        assert [float(st.V[l][P + i, 1, 3]) for i in range(3)] == [-100 * l - 0, -100 * l - 2, -100 * l - 5]
    assert [float(st.feat[P + i, 0]) for i in range(3)] == [0.0, 2.0, 5.0]


def test_draft_block_internal_consistency(tiny):
    """Consistency checks of the block head beside the pins below."""
    st = _fresh(tiny)
    dl = O.draft_block(tiny.sh, tiny.tw, tiny.hw, st, tiny.cfg.block_B)
    assert dl.shape == (tiny.cfg.block_B, tiny.cfg.vocab)
    # bidirectional block: changing the root token changes every slot's output
    st2 = _fresh(tiny)
    st2.root = (st.root + 1) % tiny.cfg.vocab
    dl2 = O.draft_block(tiny.sh, tiny.tw, tiny.hw, st2, tiny.cfg.block_B)
    assert all(float((dl[j] - dl2[j]).abs().max()) > 0 for j in range(tiny.cfg.block_B))
    # masked slots differ only through their rotary positions
    assert float((dl[1] - dl[2]).abs().max()) > 0


def _head_as_layer(hw):
    return {k: hw[k] for k in ("ln1", "wqkv", "wo", "ln2", "wgu", "wd")}


def test_draft_block_is_one_unmasked_decoder_layer(tiny):
    """Section 3.2 reading: the head is ONE decoder layer whose B rows see all P context keys and all B block
    keys.  The same rows pushed through decoder_layer (pinned elsewhere against library attention and cache-free
    chains) with the head's weights and an all-ones mask must give the same logits."""
    st = _fresh(tiny)
    sh, B, P = tiny.sh, tiny.cfg.block_B, st.P
    dl = O.draft_block(sh, tiny.tw, tiny.hw, st, B)
    X = tiny.hw["mask_embed"][None, :].repeat(B, 1)
    X[0] = tiny.tw["embed"][st.root]
    Kc, Vc = st.hK.clone(), st.hV.clone()
    pos = torch.arange(P, P + B)
    y = O.decoder_layer(sh, _head_as_layer(tiny.hw), X, pos, Kc, Vc, pos, torch.ones(B, P + B, dtype=torch.bool))
    ref = O.rmsnorm(y, tiny.hw["final_norm"], sh.rms_eps) @ tiny.tw["lm_head"].T
    assert float((dl - ref).abs().max()) <= 1e-5 * float(ref.abs().max())
    # and the pass must not have touched the committed head context
    assert torch.equal(st.hK[:P], Kc[:P]) and torch.equal(st.hV[:P], Vc[:P])


def test_draft_block_identity_layer_closed_form(tiny):
    """With W_o = 0 and W_down = 0 the layer is the identity: logits = lm_head . rmsnorm(input), written out in
    float64.  Slot 0 comes from E[root], every other slot from the mask embedding (so they are all equal)."""
    st = _fresh(tiny)
    sh, B = tiny.sh, tiny.cfg.block_B
    hw = dict(tiny.hw)
    hw["wo"] = torch.zeros_like(hw["wo"])
    hw["wd"] = torch.zeros_like(hw["wd"])
    dl = O.draft_block(sh, tiny.tw, hw, st, B).double().numpy()
    g = hw["final_norm"].double().numpy()
    W = tiny.tw["lm_head"].double().numpy()

    def closed(x):
        x = x.double().numpy()
        return W @ (x / np.sqrt(np.mean(x * x) + sh.rms_eps) * g)

    ref0, ref1 = closed(tiny.tw["embed"][st.root]), closed(hw["mask_embed"])
    scale = max(np.abs(ref0).max(), np.abs(ref1).max())
    assert np.abs(dl[0] - ref0).max() <= 1e-5 * scale
    for j in range(1, B):
        assert np.abs(dl[j] - ref1).max() <= 1e-5 * scale


def test_draft_block_single_key_closed_form(tiny):
    """B = 1 with no context: the softmax runs over one key, so the attention output is that row's own value
    vector (kv head h // G for q head h) and the whole pass has a closed form, written out in float64 numpy."""
    sh = tiny.sh
    hw, tw = tiny.hw, tiny.tw
    root = 7
    Hq, Hkv, d, F = sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.ffn
    st = O.SeqState(0, root, [], [], torch.zeros(4, Hkv, d), torch.zeros(4, Hkv, d), torch.zeros(4, sh.hidden))
    dl = O.draft_block(sh, tw, hw, st, 1).double().numpy()[0]

    def norm(x, g):
        return x / np.sqrt(np.mean(x * x) + sh.rms_eps) * g.double().numpy()

    x = tw["embed"][root].double().numpy()
    Wqkv = hw["wqkv"].double().numpy()
    v = (Wqkv[(Hq + Hkv) * d:] @ norm(x, hw["ln1"])).reshape(Hkv, d)          # value rows follow the q and k rows
    o = np.concatenate([v[h // (Hq // Hkv)] for h in range(Hq)])                # one key: softmax weight 1
    x = x + hw["wo"].double().numpy() @ o
    gu = hw["wgu"].double().numpy() @ norm(x, hw["ln2"])
    gate, up = gu[:F], gu[F:]
    x = x + hw["wd"].double().numpy() @ (gate / (1.0 + np.exp(-gate)) * up)
    ref = tw["lm_head"].double().numpy() @ norm(x, hw["final_norm"])
    assert np.abs(dl - ref).max() <= 1e-4 * np.abs(ref).max()


def test_head_context_kv_stated_reading_in_float64(tiny):
    """The head's context keys/values for committed positions (Section 3.2: they are the target's hidden states, read
    here as projections of the normalised features through the head layer's own W_k / W_v): written out row by row
    in float64 numpy with a NON-unit context gain,
        K[p] = rotate(W_k (f_p / rms(f_p) * g_ctx), p),     V[p] = W_v (f_p / rms(f_p) * g_ctx)   (not rotated).
    Dropping the norm, the gain or the key rotation, rotating the values, or reading the q rows of W_qkv instead of
    the k / v rows moves the result by O(1) of its scale; the pin allows 1e-4."""
    sh = tiny.sh
    Hq, Hkv, d, H = sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.hidden
    half = d // 2
    rng = np.random.default_rng(41)
    hw = dict(tiny.hw)
    g_ctx = rng.uniform(0.5, 1.5, size=H)
    hw["ctx_norm"] = torch.from_numpy(g_ctx).float()
    n = 5
    feats = torch.from_numpy(rng.normal(0.0, 3.0, size=(n, H))).float()       # far from unit rms: the norm matters
    pos = torch.tensor([0, 3, 17, 300, 1234])
    K, V = O.head_context_kv(sh, hw, feats, pos)
    assert K.shape == (n, Hkv, d) and V.shape == (n, Hkv, d)
    Wqkv = hw["wqkv"].double().numpy()
    Wk, Wv = Wqkv[Hq * d:(Hq + Hkv) * d], Wqkv[(Hq + Hkv) * d:]
    inv_freq = np.array([sh.rope_theta ** (-(2.0 * i) / d) for i in range(half)])
    g64 = hw["ctx_norm"].double().numpy()
    for r in range(n):
        f = feats[r].double().numpy()
        hn = f / np.sqrt(np.mean(f * f) + sh.rms_eps) * g64
        k = (Wk @ hn).reshape(Hkv, d)
        v = (Wv @ hn).reshape(Hkv, d)
        ang = float(pos[r]) * inv_freq
        c, s_ = np.cos(ang), np.sin(ang)
        k_rot = np.concatenate([k[:, :half] * c - k[:, half:] * s_, k[:, half:] * c + k[:, :half] * s_], axis=1)
        assert np.abs(K[r].double().numpy() - k_rot).max() <= 1e-4 * np.abs(k_rot).max()
        assert np.abs(V[r].double().numpy() - v).max() <= 1e-4 * np.abs(v).max()
        # the pin has teeth: each plausible mistake is far outside the allowance
        if r > 0:
            assert np.abs(k - k_rot).max() > 1e-2 * np.abs(k_rot).max()                        # rotation dropped
        no_gain = (Wv @ (f / np.sqrt(np.mean(f * f) + sh.rms_eps))).reshape(Hkv, d)
        assert np.abs(no_gain - v).max() > 1e-2 * np.abs(v).max()                              # gain dropped
        no_norm = (Wv @ (f * g64)).reshape(Hkv, d)
        assert np.abs(no_norm - v).max() > 1e-1 * np.abs(v).max()                              # norm dropped


def test_prefill_and_commit_store_head_context_kv_of_the_tapped_features(tiny):
    """The state a round leaves is this function applied to the stored features: after prefill and after rounds,
    hK / hV of every committed position equal head_context_kv(feat[p], p)."""
    st = _fresh(tiny)
    for _ in range(3):
        O.spec_round(tiny.sh, tiny.tw, tiny.hw, st, tiny.cfg.block_B, tiny.cfg.topk, tiny.cfg.tree_N)
    P = st.P
    K, V = O.head_context_kv(tiny.sh, tiny.hw, st.feat[:P], torch.arange(P))
    assert torch.allclose(st.hK[:P], K, atol=1e-6) and torch.allclose(st.hV[:P], V, atol=1e-6)


def test_draft_block_context_order_invariance(tiny):
    """No mask inside [context ; block]: permuting the context rows (keys and values together) changes nothing,
    while breaking the pairing of keys and values does."""
    st = _fresh(tiny)
    sh, B, P = tiny.sh, tiny.cfg.block_B, st.P
    dl = O.draft_block(sh, tiny.tw, tiny.hw, st, B)
    perm = torch.randperm(P, generator=torch.Generator().manual_seed(3))
    st2 = _fresh(tiny)
    st2.hK[:P] = st.hK[:P][perm]
    st2.hV[:P] = st.hV[:P][perm]
    dl2 = O.draft_block(sh, tiny.tw, tiny.hw, st2, B)
    assert float((dl - dl2).abs().max()) <= 2e-5 * float(dl.abs().max())
    st3 = _fresh(tiny)
    st3.hK[:P] = torch.roll(st.hK[:P], 1, 0)        # keys and values no longer paired
    dl3 = O.draft_block(sh, tiny.tw, tiny.hw, st3, B)
    assert float((dl - dl3).abs().max()) > 1e-4 * float(dl.abs().max())


# ------------------------------------------------------------------ multi-layer, multi-tap head

@pytest.fixture(scope="module")
def tiny2():
    """The tiny configuration with a two-layer head: head layer 0 taps target layer 0, head layer 1 taps layer 1."""
    torch.manual_seed(0)
    cfg = synth.CONFIGS["tiny"].replace(head_taps=(0, 1))
    tw_b, hw_b = synth.make_weights(cfg)
    img, ids = synth.make_context(cfg)
    t = Tiny()
    t.cfg, t.sh = cfg, O.Shape.of(cfg)
    t.tw, t.hw = O.widen(tw_b), O.widen(hw_b)
    t.ctx = O.context_embeddings(t.tw, img, ids.numpy())
    t.n_new = 40
    t.Y, t.margins = O.greedy_ar_cachefree(t.sh, t.tw, t.ctx, t.n_new)
    t.cap = cfg.ctx + t.n_new + cfg.tree_N + 64
    return t


def test_head_taps_are_the_named_target_layers(tiny2):
    """The features a head layer reads are the residual stream after the target layer it taps: equal to the output
    of a cache-free causal forward through the target truncated after that layer."""
    st = _fresh(tiny2)
    P = st.P
    for i, t in enumerate(tiny2.sh.taps):
        sh_t = O.Shape(t + 1, *[getattr(tiny2.sh, f) for f in ("hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab")])
        tw_t = dict(tiny2.tw, layers=tiny2.tw["layers"][:t + 1])
        _, feats = O.full_causal_forward(sh_t, tw_t, tiny2.ctx)
        got = st.feat if i == 0 else st.feat_more[i - 1]
        assert float((got[:P] - feats).abs().max()) <= 1e-5 * float(feats.abs().max())
    assert not torch.equal(st.feat[:P], st.feat_more[0][:P])


def test_multilayer_head_is_a_stack_of_unmasked_decoder_layers(tiny2):
    """Each head layer is one decoder layer over the block rows whose context keys/values are that layer's own
    projections of its tap: the block pushed through decoder_layer once per head layer gives the same logits."""
    st = _fresh(tiny2)
    sh, B, P = tiny2.sh, tiny2.cfg.block_B, st.P
    dl = O.draft_block(sh, tiny2.tw, tiny2.hw, st, B)
    X = tiny2.hw["mask_embed"][None, :].repeat(B, 1)
    X[0] = tiny2.tw["embed"][st.root]
    pos = torch.arange(P, P + B)
    for i in range(2):
        lw = O.head_layer(tiny2.hw, i)
        Kc = (st.hK if i == 0 else st.hK_more[i - 1]).clone()
        Vc = (st.hV if i == 0 else st.hV_more[i - 1]).clone()
        X = O.decoder_layer(sh, {k: lw[k] for k in ("ln1", "wqkv", "wo", "ln2", "wgu", "wd")}, X, pos, Kc, Vc, pos,
                            torch.ones(B, P + B, dtype=torch.bool))
    ref = O.rmsnorm(X, tiny2.hw["final_norm"], sh.rms_eps) @ tiny2.tw["lm_head"].T
    assert float((dl - ref).abs().max()) <= 1e-5 * float(ref.abs().max())
    # the second layer matters, and so does which tap feeds it
    one = O.draft_block(O.Shape.of(tiny2.cfg.replace(head_taps=(0,))), tiny2.tw, tiny2.hw, st, B)
    assert float((dl - one).abs().max()) > 1e-3 * float(dl.abs().max())


def test_explicit_last_layer_tap_is_the_one_layer_head(tiny):
    """head_taps = (n_layers - 1,) spelled out is the default one-layer head, bit for bit."""
    cfg = tiny.cfg.replace(head_taps=(tiny.cfg.n_layers - 1,))
    sh = O.Shape.of(cfg)
    st_a, st_b = _fresh(tiny), O.prefill(sh, tiny.tw, tiny.hw, tiny.ctx, tiny.cap)
    assert torch.equal(st_a.hK, st_b.hK) and torch.equal(st_a.feat, st_b.feat)
    assert torch.equal(O.draft_block(tiny.sh, tiny.tw, tiny.hw, st_a, cfg.block_B),
                       O.draft_block(sh, tiny.tw, tiny.hw, st_b, cfg.block_B))


def test_multilayer_head_rounds_lossless_and_state_equals_fresh_prefill(tiny2):
    """Rounds with the two-layer head stay lossless (Theorem 1), and the lazily appended head state of BOTH layers
    (features, keys, values of the committed positions) equals what a fresh prefill of the same tokens builds."""
    st, acc = _run_rounds(tiny2, lambda st, Y: None, 6)
    x = torch.cat([tiny2.ctx, tiny2.tw["embed"][torch.tensor(st.tokens)]], dim=0)
    ref = O.prefill(tiny2.sh, tiny2.tw, tiny2.hw, x, tiny2.cap)
    assert ref.P == st.P and ref.root == st.root
    for a, b in ((st.hK, ref.hK), (st.hV, ref.hV), (st.feat, ref.feat), (st.hK_more[0], ref.hK_more[0]),
                 (st.hV_more[0], ref.hV_more[0]), (st.feat_more[0], ref.feat_more[0])):
        assert float((a[:st.P] - b[:st.P]).abs().max()) < 1e-4 * max(1.0, float(b[:st.P].abs().max()))


# ------------------------------------------------------------------ sampling mode

def test_philox_known_answers():
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_known_answers.txt")
    n = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        got = O.philox4x32(([w[0]], [w[1]], [w[2]], [w[3]]), (w[4], w[5]))[:, 0]
        assert [int(x) for x in got] == w[6:10]
        n += 1
    assert n == 3


def test_uniform_field_layout_and_range():
    seed, pos, V = 0x1234567890ABCDEF, 777, 1003
    u = O.uniform_field(seed, pos, V)
    assert u.dtype == np.float32 and u.shape == (V,)
    assert float(u.min()) > 0.0 and float(u.max()) < 1.0
    # id 4b + j reads word j of the block whose counter is (b, position, 0, 0)
    for v in (0, 1, 6, 1002):
        w = O.philox4x32(([v // 4], [pos], [0], [0]), (seed & 0xFFFFFFFF, seed >> 32))[v % 4, 0]
        assert u[v] == np.float32(((int(w) >> 9) + 0.5) * 2.0 ** -23)
    # another position or seed gives another field
    assert not np.array_equal(u, O.uniform_field(seed, pos + 1, V))
    assert not np.array_equal(u, O.uniform_field(seed + 1, pos, V))


def test_gumbel_max_draws_follow_the_softmax():
    """Frequencies of arg-max(logits + g) over many positions against softmax(logits): chi-square, 7 degrees of
    freedom, and the same at temperature 2 (inv_temperature 0.5)."""
    logits = torch.tensor([[2.0, 1.0, 0.5, 0.0, -0.5, -1.0, 1.5, -3.0]])
    n = 20000
    for inv_t in (1.0, 0.5):
        p = torch.softmax(logits[0] * inv_t, dim=0).numpy()
        ids, _ = O.sample_rows(logits.repeat(n, 1), list(range(n)), seed=99, inv_temperature=inv_t)
        cnt = np.bincount(ids, minlength=8)
        chi2 = float(((cnt - n * p) ** 2 / (n * p)).sum())
        assert chi2 < 24.3, (inv_t, chi2, cnt)          # P(chi2_7 > 24.3) = 0.001


def test_sampled_rounds_equal_plain_ancestral_sampling(tiny):
    """Sampling walk: tree rounds commit exactly the tokens that plain ancestral sampling (one cache-free forward
    per token) draws with the same noise field, whatever the trees are."""
    seed = 0xC0FFEE
    st = _fresh(tiny)
    first, P0 = st.root, st.P
    rng = np.random.default_rng(17)
    n_rounds = 6
    ref = O.sampled_ar_cachefree(tiny.sh, tiny.tw, tiny.ctx, first, n_rounds * tiny.cfg.block_B, seed)
    accepted = []
    for r in range(n_rounds):
        done = st.P - P0                      # tokens committed after the first root so far
        Y = ref[done:done + tiny.cfg.L]
        tree = None
        if r % 2 == 1:                        # every other round: a random tree with the true draws planted
            def pref(parent, depth):
                return int(Y[depth - 1]) if rng.random() < 0.8 else None
            tok, par, dep = synth.random_tree(8, tiny.cfg.L, tiny.cfg.vocab, rng, tokens_for=pref)
            tok[0] = st.root
            tree = O.tree_from_arrays(tok, par, dep, N=8)
        info = O.spec_round_sampled(tiny.sh, tiny.tw, tiny.hw, st, tiny.cfg.block_B, tiny.cfg.topk, tiny.cfg.tree_N,
                                    seed, tree=tree)
        accepted.append(info["a"])
        assert float(np.min(info["margins"][:info["tree"].n_nodes])) > 1e-4, "near-tie in a perturbed row: pick another seed"
    committed = st.tokens + [st.root]
    assert committed[0] == first
    assert committed[1:] == ref[:len(committed) - 1]
    assert sum(accepted) > 0


def test_root_entropy_closed_forms():
    """Entropy of the root row (Section 4) against closed forms: uniform, two-level and shifted distributions."""
    V = 1000
    assert abs(O.root_entropy(torch.zeros(V)) - math.log(V)) < 1e-9
    assert abs(O.root_entropy(torch.full((V,), 3.7)) - math.log(V)) < 1e-9          # a constant shift changes nothing
    # one token with probability q, the rest uniform: H = -q log q - (1-q) log((1-q)/(V-1))
    for q in (0.5, 0.9, 0.999):
        x = torch.zeros(V, dtype=torch.float64)
        x[17] = math.log(q / ((1 - q) / (V - 1)))
        ref = -q * math.log(q) - (1 - q) * math.log((1 - q) / (V - 1))
        assert abs(O.root_entropy(x) - ref) < 1e-9
    # a dominant logit: H -> 0; and H never exceeds log V
    x = torch.randn(V, generator=torch.Generator().manual_seed(1))
    assert 0.0 < O.root_entropy(x) < math.log(V)
    x[3] = 80.0
    assert O.root_entropy(x) < 1e-20 + 1e-12


def test_controlled_match_acceptance_statistics(tiny):
    """Measured mean accepted length under controlled per-depth match probability sits on Eq. 2."""
    rng = np.random.default_rng(21)
    cfg = tiny.cfg
    L, k, p = 15, 8, 0.8
    lp = synth.controlled_marginals(p, k, L)
    Y = list(np.random.default_rng(5).integers(0, 50000, size=L + 1))
    acc = []
    for _ in range(600):
        ids = synth.controlled_candidates(Y[:L], p, k, L, 50000, rng)
        tree = O.build_tree(1, ids, lp, 64)
        acc.append(O.accepted_length_bruteforce(tree, Y))
    mean, sd = np.mean(acc), np.std(acc) / math.sqrt(len(acc))
    # the rank-0 chain reaches depth 15 inside a 64-node tree at p = 0.8
    assert abs(mean - O.expected_accept(p, L)) < 4 * sd + 0.05
