"""GPU parity tests: the CUDA library, called through its C ABI, against the CPU oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import glance_oracle as O
from paper_2609_00355_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def harness():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from tests import parity_harness
    return parity_harness


@pytest.fixture(scope="module")
def tiny_run(harness):
    return harness.ParityRun(synth.CONFIGS["tiny"])


def make_engine(cfg, batch=1, max_len=None):
    """An engine on random weights without any oracle state (kernel-level tests)."""
    from paper_2609_00355_b200.binding import Engine
    tw, hw = synth.make_weights(cfg, "cuda")
    return Engine(cfg, tw, hw, batch=batch, max_len=max_len)


# ------------------------------------------------------------------ GEMM alone

@pytest.fixture(scope="module")
def gemm_eng(harness):
    return make_engine(synth.CONFIGS["tiny"].replace(tree_N=128, vocab=256), batch=2)


TC_SHAPES = [(256, 256, 8, 1), (512, 256, 64, 2), (1408, 256, 16, 1), (1000, 704, 37, 3), (4608, 3584, 64, 4),
             (3584, 18944, 64, 5), (640, 1024, 128, 4), (130, 64, 1, 1), (384, 512, 200, 2), (37888, 3584, 64, 1)]


@pytest.mark.parametrize("Nout,K,R,S", TC_SHAPES)
def test_gemm_tc_planes(gemm_eng, Nout, K, R, S):
    """Weight-streaming GEMM, fp32 split-K planes, against an fp64 matmul of the same bf16 inputs."""
    eng = gemm_eng
    g = torch.Generator(device="cuda").manual_seed(Nout + K + R)
    W = (torch.randn(Nout, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    X = torch.randn(R, K, generator=g, device="cuda").to(torch.bfloat16)
    Y = torch.full((S, R, Nout), float("nan"), device="cuda")
    eng.glance_debug_gemm(0, W, X, Y=Y, S=S)
    assert eng.glance_poll_status() == 0
    ref = X.double() @ W.double().T
    got = Y.double().sum(0)
    assert float((got - ref).abs().max()) <= 1e-4 * float(ref.abs().max()) + 1e-5
    Y2 = torch.zeros_like(Y)
    eng.glance_debug_gemm(0, W, X, Y=Y2, S=S)
    assert torch.equal(Y, Y2)


def test_bounded_wait_runs_out_and_the_context_stays_usable(gemm_eng):
    """Failure detection on the device, without a fault: one ring slot of a tiny GEMM is never filled (chosen on the
    host), the MMA issuer's bounded wait on it gives up after 100 us, the CTA drains the copies it has in flight,
    frees its tensor memory and returns; the host reads GLANCE_E_TIMEOUT, and the next launch is correct."""
    eng = gemm_eng
    g = torch.Generator(device="cuda").manual_seed(99)
    W = (torch.randn(128, 512, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    X = torch.randn(16, 512, generator=g, device="cuda").to(torch.bfloat16)
    ref = X.double() @ W.double().T
    for kstep in (2, 6):                                   # inside the first ring fill, and in a re-used slot
        Y = torch.zeros(1, 16, 128, device="cuda")
        eng.glance_debug_stall_next_gemm(kstep, 100_000)
        eng.glance_debug_gemm(0, W, X, Y=Y, S=1)
        assert eng.glance_poll_status() == -5              # GLANCE_E_TIMEOUT
        assert eng.glance_poll_status() == 0               # cleared by the read
        # the hook was one shot: the same launch again is a normal one
        Y2 = torch.full((1, 16, 128), float("nan"), device="cuda")
        eng.glance_debug_gemm(0, W, X, Y=Y2, S=1)
        assert eng.glance_poll_status() == 0
        assert float((Y2[0].double() - ref).abs().max()) <= 1e-4 * float(ref.abs().max()) + 1e-5


@pytest.mark.parametrize("F,K,R", [(704, 256, 8), (2816, 1024, 32), (18944, 3584, 64), (320, 128, 130)])
def test_gemm_tc_swiglu(gemm_eng, F, K, R):
    eng = gemm_eng
    g = torch.Generator(device="cuda").manual_seed(F + K + R)
    W = (torch.randn(2 * F, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    X = torch.randn(R, K, generator=g, device="cuda").to(torch.bfloat16)
    act = torch.full((R, F), float("nan"), dtype=torch.bfloat16, device="cuda")
    eng.glance_debug_gemm(1, W, X, act=act)
    assert eng.glance_poll_status() == 0
    gu = X.double() @ W.double().T
    ref = torch.nn.functional.silu(gu[:, :F]) * gu[:, F:]
    assert float((act.double() - ref).abs().max()) <= 1e-2 * float(ref.abs().max())


@pytest.mark.parametrize("V,K,R", [(1024, 256, 8), (32000, 1024, 32), (152064, 3584, 64), (1000, 128, 129)])
def test_gemm_tc_argmax(gemm_eng, V, K, R):
    eng = gemm_eng
    g = torch.Generator(device="cuda").manual_seed(V + K + R)
    W = (torch.randn(V, K, generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    X = torch.randn(R, K, generator=g, device="cuda").to(torch.bfloat16)
    W[7] = W[V - 3]                                       # an exact tie between two ids: the lower one must win
    X[0] = W[7] * 4
    am = torch.full((R,), -1, dtype=torch.int32, device="cuda")
    Y = torch.full((R, V), float("nan"), device="cuda")
    for rep in range(2):                                  # second call checks that keys and counter were re-armed
        eng.glance_debug_gemm(2, W, X, Y=Y, argmax=am)
        assert eng.glance_poll_status() == 0
        ref = X.double() @ W.double().T
        assert float((Y.double() - ref).abs().max()) <= 1e-4 * float(ref.abs().max()) + 1e-5
        # the arg-max is taken on the kernel's own fp32 accumulators, ties to the lowest id
        assert np.array_equal(am.cpu().numpy(), O.argmax_lowest(Y.cpu()))
        assert int(am[0]) == 7
    am2 = torch.full((R,), -1, dtype=torch.int32, device="cuda")
    eng.glance_debug_gemm(2, W, X, argmax=am2)          # without the debug logits
    assert torch.equal(am, am2)


# ------------------------------------------------------------------ attention alone

def _fill_cache(eng, seq, layer, K, V):
    """Write logical rows K,V [n,Hkv,d] of one sequence/layer into the paged pool."""
    page = eng.cfg.page_size
    n = K.shape[0]
    pos = torch.arange(n, device=eng.device)
    pages = eng.page_table[seq].long()[pos // page]
    eng.kv_pool[layer, pages, 0, :, pos % page, :] = K.to(torch.bfloat16)
    eng.kv_pool[layer, pages, 1, :, pos % page, :] = V.to(torch.bfloat16)


def test_attention_mask_bits_one_hot(harness):
    """Every (row, key) mask bit changes the output by O(1): tree keys dominate, values are one-hot."""
    cfg = synth.CONFIGS["tiny"].replace(tree_N=64, vocab=256, n_layers=2)
    eng = make_engine(cfg, max_len=320)
    rng = np.random.default_rng(3)
    N, Hq, Hkv, d = 64, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    for P in (0, 3, 64, 70):
        tok, par, dep = synth.random_tree(N, 15, 1000, rng)
        tree = O.tree_from_arrays(tok, par, dep)
        n = P + N
        # context keys score 0, tree key j scores 5 on every query (q = 1): visible tree keys dominate the
        # softmax, and value j is one-hot at dim j mod d, so each output dim reports one tree key's weight
        K = torch.zeros(n, Hkv, d)
        V = torch.zeros(n, Hkv, d)
        for j in range(P, n):
            K[j, :, j % d] = 5.0 * math.sqrt(d)
            V[j, :, j % d] = 1.0
        V[:P, :, 0] = -1.0
        q = torch.ones(N, Hq, d)
        eng.seq_len[0] = P
        # poison the rows after the last key: they must never contribute
        Kp = torch.cat([K, torch.full((8, Hkv, d), float("nan"))])
        Vp = torch.cat([V, torch.full((8, Hkv, d), float("nan"))])
        _fill_cache(eng, 0, 1, Kp.cuda(), Vp.cuda())
        out = torch.zeros(N, Hq * d, dtype=torch.bfloat16, device="cuda")
        anc = torch.from_numpy(tree.anc.view(np.int64)).cuda()[None].contiguous()
        eng.glance_debug_attention(1, q.to(torch.bfloat16).cuda().reshape(N, Hq * d).contiguous(), anc, N, out)
        eng.check_device_status()
        vis = O.visibility(tree, P)
        ref = O.attention(q, K, V, vis)
        got = out.float().cpu().reshape(N, Hq, d)
        assert torch.isfinite(got).all()
        assert float((got - ref).abs().max()) < 0.01
        # any single flipped tree-key bit would move the reference by far more than the tolerance
        for (i, j) in [(N - 1, 1), (5, 5), (17, 3), (40, 40)]:
            m2 = vis.clone()
            m2[i, P + j] = ~m2[i, P + j]
            if m2[i, P:].any():
                assert float((O.attention(q, K, V, m2) - ref).abs().max()) > 0.04


@pytest.mark.parametrize("name,P,T", [("tiny", 300, 8), ("small", 704, 32), ("7b", 1536, 64), ("7b", 100, 128),
                                      ("long", 8704, 128), ("7b", 0, 64), ("7b", 1, 1), ("tiny", 63, 2),
                                      ("7b", 191, 16), ("7b", 449, 33), ("7b", 3000, 64), ("small", 65, 32)])
def test_attention_random_inputs(harness, name, P, T):
    base = synth.CONFIGS[name]
    cfg = base.replace(n_layers=1, vocab=256, ffn=64, hidden=64, tree_N=T, n_img=2, n_txt=1, rounds=1)
    eng = make_engine(cfg, batch=2, max_len=P + T + 64)
    rng = np.random.default_rng(P + T)
    g = torch.Generator().manual_seed(P)
    Hq, Hkv, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    Ps = [P, max(1, P // 3)]
    qs, refs, ancs = [], [], []
    for s in range(2):
        tok, par, dep = synth.random_tree(T, 15, 1000, rng)
        tree = O.tree_from_arrays(tok, par, dep)
        K = torch.randn(Ps[s] + T, Hkv, d, generator=g).to(torch.bfloat16)
        V = torch.randn(Ps[s] + T, Hkv, d, generator=g).to(torch.bfloat16)
        q = (torch.randn(T, Hq, d, generator=g) * 1.5).to(torch.bfloat16)
        eng.seq_len[s] = Ps[s]
        # the rest of the last page holds NaN bits: rows after the last key must never contribute
        pad = (-(Ps[s] + T)) % cfg.page_size
        poison = torch.full((pad, Hkv, d), float("nan"), dtype=torch.bfloat16)
        _fill_cache(eng, s, 0, torch.cat([K, poison]).cuda(), torch.cat([V, poison]).cuda())
        refs.append(O.attention(q.float(), K.float(), V.float(), O.visibility(tree, Ps[s])))
        qs.append(q.reshape(T, Hq * d))
        ancs.append(torch.from_numpy(tree.anc.view(np.int64)))
    out = torch.zeros(2 * T, Hq * d, dtype=torch.bfloat16, device="cuda")
    eng.glance_debug_attention(0, torch.cat(qs).cuda().contiguous(), torch.stack(ancs).cuda().contiguous(), T, out)
    eng.check_device_status()
    out2 = torch.zeros_like(out)
    eng.glance_debug_attention(0, torch.cat(qs).cuda().contiguous(), torch.stack(ancs).cuda().contiguous(), T, out2)
    assert torch.equal(out, out2)                       # split merge is order-fixed: run-to-run identical
    assert torch.isfinite(out.float()).all()
    for s in range(2):
        got = out[s * T:(s + 1) * T].float().cpu().reshape(T, Hq, d)
        assert float((got - refs[s]).abs().max()) <= 2e-2 * float(refs[s].abs().max())
    # no mask = every extra key visible (the draft block's bidirectional attention)
    eng.glance_debug_attention(0, torch.cat(qs).cuda().contiguous(), None, T, out)
    for s in range(2):
        full = torch.ones(T, Ps[s] + T, dtype=torch.bool)
        Kf, Vf = eng.gather_kv(s, 0, Ps[s] + T)
        ref = O.attention(qs[s].float().reshape(T, Hq, d), Kf.float().cpu(), Vf.float().cpu(), full)
        got = out[s * T:(s + 1) * T].float().cpu().reshape(T, Hq, d)
        assert float((got - ref).abs().max()) <= 2e-2 * float(ref.abs().max())


def test_attention_two_term_queries_and_outputs(harness):
    """fp32 queries given as two bf16 terms, outputs read back as two terms: the only roundings left inside the
    kernel are those of the probabilities and the fp32 accumulation, so the error against the oracle must sit far
    below the one-term path's, whose queries alone are off by 2^-9."""
    cfg = synth.CONFIGS["7b"].replace(n_layers=1, vocab=256, ffn=64, hidden=64, tree_N=64, n_img=2, n_txt=1, rounds=1)
    P, T = 1536, 64
    eng = make_engine(cfg, batch=1, max_len=P + T + 64)
    rng = np.random.default_rng(17)
    g = torch.Generator().manual_seed(17)
    Hq, Hkv, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    tok, par, dep = synth.random_tree(T, 15, 1000, rng)
    tree = O.tree_from_arrays(tok, par, dep)
    K = (torch.randn(P + T, Hkv, d, generator=g) * 1.2).to(torch.bfloat16)
    V = (torch.randn(P + T, Hkv, d, generator=g) * 1.2).to(torch.bfloat16)
    q = torch.randn(T, Hq, d, generator=g) * 1.2                     # fp32: not representable in one bf16 term
    eng.seq_len[0] = P
    _fill_cache(eng, 0, 0, K.cuda(), V.cuda())
    ref = O.attention(q, K.float(), V.float(), O.visibility(tree, P))
    q_hi = q.to(torch.bfloat16)
    q_lo = (q - q_hi.float()).to(torch.bfloat16)
    anc = torch.from_numpy(tree.anc.view(np.int64)).cuda()[None].contiguous()

    def run(lo):
        out = torch.zeros(T, Hq * d, dtype=torch.bfloat16, device="cuda")
        out_lo = torch.zeros_like(out)
        eng.glance_debug_attention(0, q_hi.reshape(T, Hq * d).cuda().contiguous(), anc, T, out,
                                   q_lo=lo.reshape(T, Hq * d).cuda().contiguous() if lo is not None else None, out_lo=out_lo)
        eng.check_device_status()
        got = (out.float() + out_lo.float()).cpu().reshape(T, Hq, d)
        return float((got - ref).pow(2).mean().sqrt()), float((got - ref).abs().max())

    rms1, max1 = run(None)
    rms2, max2 = run(q_lo)
    scale = float(ref.abs().max())
    print(f"one-term q: rms {rms1:.3e} max {max1:.3e}; two-term q: rms {rms2:.3e} max {max2:.3e}; scale {scale:.3f}")
    assert max2 <= 1e-2 * scale
    assert rms2 < 0.75 * rms1                                        # the second term removes the queries' share


# ------------------------------------------------------------------ tree builder (bit-exact)

@pytest.mark.parametrize("name", ["tiny", "small", "7b", "long"])
def test_build_tree_bit_exact(harness, tiny_run, name):
    base = synth.CONFIGS[name]
    cfg = synth.CONFIGS["tiny"].replace(block_B=base.block_B, topk=base.topk, tree_N=base.tree_N, n_img=2, n_txt=1,
                                        rounds=1, vocab=256)
    eng = make_engine(cfg, batch=3)
    rng = np.random.default_rng(17)
    L, k, N = cfg.L, cfg.topk, cfg.tree_N
    for trial in range(6):
        ids = np.zeros((3, L, k), dtype=np.int32)
        lp = np.zeros((3, L, k), dtype=np.float32)
        for s in range(3):
            if trial % 3 == 2:
                lp[s] = synth.controlled_marginals([0.3, 0.6, 0.9][s], k, L)
                ids[s] = rng.integers(0, 1000, size=(L, k))
            else:
                ids[s], lp[s] = synth.random_topk(L, k, 1000, rng, ties=(trial % 3 == 1))
        roots = torch.tensor([5, 6, 7], dtype=torch.int32, device="cuda")
        eng.glance_build_tree(torch.from_numpy(ids).cuda(), torch.from_numpy(lp).cuda(), root=roots)
        eng.check_device_status()
        for s in range(3):
            harness.assert_tree_bits(harness.tree_from_device(eng.tree, s), O.build_tree(5 + s, ids[s], lp[s], N))


@pytest.mark.parametrize("block_B,topk,tree_N", [(4, 1, 8), (3, 2, 16), (2, 3, 8), (5, 1, 128), (3, 3, 100)])
def test_build_tree_exhausted_frontier_bit_exact(harness, block_B, topk, tree_N):
    """Budgets the candidate trie cannot fill (sum_l k^l < N - 1): the frontier runs empty, n_nodes < N, and the
    rows from n_nodes on are padding (token 0, parent -1, visible to themselves only) -- all bit for bit."""
    cfg = synth.CONFIGS["tiny"].replace(block_B=block_B, topk=topk, tree_N=tree_N, n_img=2, n_txt=1, rounds=1, vocab=256)
    eng = make_engine(cfg, batch=2)
    rng = np.random.default_rng(23)
    L, k, N = cfg.L, cfg.topk, cfg.tree_N
    prefixes = sum(k ** l for l in range(1, L + 1))
    assert prefixes < N - 1
    for trial in range(4):
        ids = np.zeros((2, L, k), dtype=np.int32)
        lp = np.zeros((2, L, k), dtype=np.float32)
        for s in range(2):
            ids[s], lp[s] = synth.random_topk(L, k, 1000, rng, ties=(trial % 2 == 1))
        roots = torch.tensor([5, 6], dtype=torch.int32, device="cuda")
        eng.glance_build_tree(torch.from_numpy(ids).cuda(), torch.from_numpy(lp).cuda(), root=roots)
        eng.check_device_status()
        for s in range(2):
            got = harness.tree_from_device(eng.tree, s)
            want = O.build_tree(5 + s, ids[s], lp[s], N)
            assert want.n_nodes == prefixes + 1
            harness.assert_tree_bits(got, want)
            assert int(eng.tree.n_nodes[s]) == prefixes + 1
            assert all(int(v) == -1 for v in eng.tree.parent[s, prefixes + 1:].cpu())


@pytest.mark.parametrize("vocab,topk,distinct", [(1000, 4, 3), (1000, 16, 2), (130, 8, 130), (8192, 16, 1), (2000, 8, 40)])
def test_draft_topk_fused_in_lm_head_with_massive_ties(harness, vocab, topk, distinct):
    """The per-offset top-k inside the LM head's epilogue under the worst ties: the LM head repeats `distinct` rows,
    so every logit value is shared by vocab / distinct ids spread over all tiles (tiles with more equal values at
    the bound than they have slots, a merge with more keys at the bound than it collects, a last tile of two
    features, k equal to the slot count).  Against the exact (logit desc, id asc) order of the library's own logits."""
    cfg = synth.CONFIGS["tiny"].replace(vocab=vocab, topk=topk, block_B=5, tree_N=8, n_img=20, n_txt=12, rounds=1)
    tw, hw = synth.make_weights(cfg, "cuda")
    tw["lm_head"] = tw["lm_head"][:distinct].repeat((vocab + distinct - 1) // distinct, 1)[:vocab].contiguous()
    from paper_2609_00355_b200.binding import Engine
    eng = Engine(cfg, tw, hw, batch=2)
    for s in range(2):
        img, ids = synth.make_context(cfg, "cuda", seed=3 + s)
        eng.prefill_context(s, img, ids % min(vocab, 1000))
    B, L = cfg.block_B, cfg.L
    for rep in range(2):                                   # the second call meets re-armed bounds and stale key slots
        logits = torch.zeros(2, B, vocab, dtype=torch.float32, device="cuda")
        eng.glance_draft_block(logits_dbg=logits)
        eng.check_device_status()
        lg = logits.cpu().numpy()
        for s in range(2):
            for j in range(1, B):
                row = lg[s, j]
                order = np.lexsort((np.arange(vocab), -row))[:topk]
                assert np.array_equal(eng.topk_ids[s, j - 1].cpu().numpy(), order.astype(np.int32)), (rep, s, j)
                lse = float(torch.logsumexp(torch.from_numpy(row).double(), dim=0))
                got = eng.topk_lp[s, j - 1].cpu().numpy().astype(np.float64)
                assert np.abs(got - (row[order].astype(np.float64) - lse)).max() < 1e-4
        eng.glance_build_tree()
        eng.glance_verify_tree()
        eng.glance_accept_commit()


# ------------------------------------------------------------------ walk + commit (bit-exact)

def test_walk_commit_examples_and_compaction_hazard(harness):
    cfg = synth.CONFIGS["tiny"]
    run = harness.ParityRun(cfg, ctx_lens=[(40, 9)])
    eng = run.eng
    ex_parent = [-1, 0, 0, 1, 1, 2, 3, 4]
    ex_depth = [0, 1, 1, 2, 2, 2, 3, 3]
    ex_token = [7, 11, 12, 21, 22, 23, 31, 32]
    tree = O.tree_from_arrays(ex_token, ex_parent, ex_depth)
    harness.tree_to_device(eng, [tree])
    cases = [([11, 22, 0, 0, 99, 0, 0, 0], (2, [0, 1, 4], [11, 22], 99)),
             ([12, 0, 23, 0, 0, 5, 0, 0], (2, [0, 2, 5], [12, 23], 5)),       # row P+2: source, then destination
             ([13, 0, 0, 0, 0, 0, 0, 0], (0, [0], [], 13)),
             ([11, 21, 0, 31, 0, 0, 44, 0], (3, [0, 1, 3, 6], [11, 21, 31], 44))]
    for am, expect in cases:
        assert O.walk(tree, np.array(am)) == expect
        P = int(eng.seq_len[0])
        # distinct recognisable bytes in every scratch row
        for i in range(8):
            pos = P + i
            pg = int(eng.page_table[0, pos // 64])
            eng.kv_pool[:, pg, :, :, pos % 64, :] = float(i + 1)
        eng.hidden.copy_(torch.arange(8, device="cuda")[None, :, None].expand_as(eng.hidden).to(torch.bfloat16))
        before = eng.kv_pool.clone()
        eng.argmax.copy_(torch.tensor([am], dtype=torch.int32))
        eng.glance_accept_commit()
        eng.check_device_status()
        a, path, out, new_root = expect
        assert int(eng.accept_len[0]) == a
        assert eng.path[0, :a + 1].tolist() == path and eng.path[0, a + 1:].tolist() == [-1] * (cfg.block_B - a - 1)
        assert eng.out_tokens[0, :a + 1].tolist() == out + [new_root]
        assert int(eng.seq_len[0]) == P + a + 1 and int(eng.root[0]) == new_root and int(eng.feat_count[0]) == a + 1
        run._check_compaction(0, P, path, before)
        assert eng.feat[0, :a + 1, 0].float().tolist() == [float(v) for v in path]


def test_commit_forced_and_bad_path_is_reported(harness):
    cfg = synth.CONFIGS["tiny"]
    run = harness.ParityRun(cfg, ctx_lens=[(20, 5)])
    eng = run.eng
    P = int(eng.seq_len[0])
    before = eng.kv_pool.clone()
    path = torch.tensor([[0, 3, 7, -1]], dtype=torch.int32, device="cuda")
    eng.glance_commit_forced(path, torch.tensor([3], dtype=torch.int32, device="cuda"),
                             torch.tensor([42], dtype=torch.int32, device="cuda"))
    eng.check_device_status()
    assert int(eng.seq_len[0]) == P + 3 and int(eng.root[0]) == 42
    run._check_compaction(0, P, [0, 3, 7], before)
    # a non-increasing path is rejected by the device-side check (status word, no fault)
    bad = torch.tensor([[0, 5, 2, -1]], dtype=torch.int32, device="cuda")
    eng.glance_commit_forced(bad, torch.tensor([3], dtype=torch.int32, device="cuda"),
                             torch.tensor([1], dtype=torch.int32, device="cuda"))
    assert eng.glance_poll_status() == -6
    assert eng.glance_poll_status() == 0


def test_profile_read_before_enable_is_a_state_error(harness):
    eng = make_engine(synth.CONFIGS["tiny"], batch=1)
    import ctypes as C
    ms, by, n = (C.c_double * 5)(), (C.c_double * 5)(), (C.c_int64 * 5)()
    assert eng.lib.glance_profile_read(eng.ctx, ms, by, n) == -7          # GLANCE_E_STATE
    assert eng.lib.glance_status_string(-7) == b"invalid call order"
    eng.glance_profile_enable(True)
    assert eng.lib.glance_profile_read(eng.ctx, ms, by, n) == 0


def test_capacity_overflow_sets_status_not_fault(harness):
    cfg = synth.CONFIGS["tiny"]
    run = harness.ParityRun(cfg, ctx_lens=[(20, 5)])
    eng = run.eng
    eng.seq_len[0] = eng.pages_per_seq * 64 - 2          # P + N exceeds the page budget
    eng.glance_verify_tree()
    assert eng.glance_poll_status() == -3                 # GLANCE_E_CAPACITY, from the row setup kernel
    assert eng.glance_poll_status() == 0


# ------------------------------------------------------------------ the whole round, stage by stage

def test_prefill_state_tiny(tiny_run):
    tiny_run.check_state()
    tiny_run.check_head_state()


def test_rounds_tiny_drafted_trees(tiny_run):
    """Tiny config, trees from the library's own draft (random head: short accepts)."""
    for _ in range(4):
        tiny_run.round()
    tiny_run.check_head_state()


def test_rounds_tiny_controlled_match(tiny_run):
    """Tiny config, 16 rounds at p_m = 0.7: accepted paths, compaction and state after every round."""
    for _ in range(16):
        tiny_run.round(p_m=0.7)
    tiny_run.check_head_state()
    st = tiny_run.stats
    print("tiny parity stats:", st)
    assert st["accepted"] > 0
    assert st["max_rel_logit"] <= 2e-2


def test_rounds_tiny_single_node_is_plain_ar(harness):
    """tree_N = 1 rounds commit exactly one token each (tau = 1) and follow the oracle's greedy stream."""
    cfg = synth.CONFIGS["tiny"].replace(tree_N=1)
    run = harness.ParityRun(cfg, ctx_lens=[(50, 14)])
    for _ in range(6):
        run.round(check_draft=False)
    assert run.stats["accepted"] == 0 and run.stats["rounds"] == 6


@pytest.mark.parametrize("p_m", [0.3, 0.6, 0.9])
def test_rounds_small(harness, p_m):
    cfg = synth.CONFIGS["small"]
    run = harness.ParityRun(cfg)
    run.check_state()
    run.check_head_state()
    for r in range(6):
        run.round(p_m=p_m, check_draft=(r < 2))
    run.check_head_state()
    print("small parity stats p_m", p_m, run.stats)
    assert run.stats["max_rel_logit"] <= 2e-2


def test_rounds_batch3_ragged(harness):
    """Three sequences with different context lengths and trees in one call (ragged accepts)."""
    cfg = synth.CONFIGS["tiny"].replace(tree_N=16, block_B=6, topk=3)
    run = harness.ParityRun(cfg, batch=3, ctx_lens=[(100, 30), (17, 3), (200, 57)])
    run.check_state()
    for _ in range(5):
        run.round(p_m=0.75)
    run.check_head_state()
    print("batch parity stats:", run.stats)


def test_round_7b_shape_one_layer_slice(harness):
    """Full 7B widths (hidden 3584, 28/4 heads of 128, FFN 18944, N 64) on 2 layers and a reduced vocabulary:
    the launch configuration of the benchmark's per-layer kernels, small enough for the oracle."""
    cfg = synth.CONFIGS["7b"].replace(n_layers=2, vocab=4096, n_img=150, n_txt=43, rounds=4)
    run = harness.ParityRun(cfg)
    run.check_state()
    for r in range(3):
        run.round(p_m=0.8, check_draft=(r == 0))
    print("7b-slice parity stats:", run.stats)


def test_round_long_shape_slice_128_rows(harness):
    """N = 128 tree rows at the full 7B widths (2 layers, reduced vocabulary): the 128-row GEMM tiles with
    two-term activations (UMMA N = 256) and the two-word ancestor masks of the long-context configuration."""
    cfg = synth.CONFIGS["long"].replace(n_layers=2, vocab=4096, n_img=300, n_txt=85, rounds=3)
    run = harness.ParityRun(cfg)
    run.check_state()
    for r in range(2):
        run.round(p_m=0.5, check_draft=(r == 0))
    print("long-slice parity stats:", run.stats)
    assert run.stats["max_rel_logit"] <= 2e-2


def test_rounds_batch3_two_row_blocks(harness):
    """Three sequences of 64 tree rows each: 192 verify rows span two 128-row blocks of every GEMM."""
    cfg = synth.CONFIGS["tiny"].replace(tree_N=64, block_B=8, topk=4)
    run = harness.ParityRun(cfg, batch=3, ctx_lens=[(90, 20), (33, 9), (150, 41)])
    run.check_state()
    for _ in range(3):
        run.round(p_m=0.7)
    run.check_head_state()
    print("batch3 x 64 rows parity stats:", run.stats)
    assert run.stats["max_rel_logit"] <= 2e-2


def test_rounds_batch16_four_row_blocks_ragged(harness):
    """Sixteen ragged sequences of 32 tree rows each: 512 verify rows = four 128-row blocks of every GEMM (the launch
    shapes of the small-batch serving configuration: split-K chosen for whole waves, two key splits in the
    attention), 256 draft rows, per-sequence trees, accepts and compaction."""
    cfg = synth.CONFIGS["tiny"].replace(tree_N=32, block_B=8, topk=3)
    rng = np.random.default_rng(12)
    ctx_lens = [(int(a), int(b)) for a, b in zip(rng.integers(5, 220, size=16), rng.integers(1, 40, size=16))]
    run = harness.ParityRun(cfg, batch=16, ctx_lens=ctx_lens)
    run.check_state()
    for r in range(2):
        run.round(p_m=(0.7 if r else None), check_draft=(r == 0))
    run.check_head_state()
    print("batch16 x 32 rows parity stats:", run.stats)
    assert run.stats["max_rel_logit"] <= 2e-2


def test_page_budget_exact_fit_passes_and_one_more_row_is_a_capacity_fault(harness):
    """seq_len + tree_N == page_size * max_pages_per_seq is legal (the last tree row sits in the last slot of the
    last page); one committed position more is reported as GLANCE_E_CAPACITY and nothing faults."""
    cfg = synth.CONFIGS["tiny"]
    run = harness.ParityRun(cfg, ctx_lens=[(20, 5)])
    eng = run.eng
    cap = eng.pages_per_seq * 64
    snap = eng.snapshot_state()
    eng.seq_len[0] = cap - cfg.tree_N                    # rows cap - N .. cap - 1: exactly fits
    eng.glance_build_tree()
    eng.glance_verify_tree()
    assert eng.glance_poll_status() == 0
    eng.seq_len[0] = cap - cfg.tree_N + 1
    eng.glance_verify_tree()
    assert eng.glance_poll_status() == -3
    eng.restore_state(snap)
    run.round(p_m=0.7)                                    # the engine is still good
    assert eng.glance_poll_status() == 0


def test_rounds_tiny_chain_k1(harness):
    """k = 1: the candidate tree degenerates to the rank-0 chain (classic chain drafting through the same path)."""
    cfg = synth.CONFIGS["tiny"].replace(topk=1, tree_N=4)
    run = harness.ParityRun(cfg)
    run.check_state()
    for r in range(6):
        run.round(p_m=0.8, check_draft=(r == 0))
    print("chain parity stats:", run.stats)
    assert run.stats["max_rel_logit"] <= 2e-2


def test_rounds_tiny_sampling_mode(harness):
    """Sampling walk at temperature 1: every row's decision is a draw (Gumbel-max over the position-keyed noise
    field); draws, walk, commit and state against the oracle's sampling rounds, with drafted and planted trees."""
    run = harness.ParityRun(synth.CONFIGS["tiny"])
    run.check_state()
    for r in range(8):
        run.round(p_m=(0.7 if r % 2 else None), check_draft=False, sample_seed=0xC0FFEE + 17)
    run.check_head_state()
    print("sampling parity stats:", run.stats)
    assert run.stats["accepted"] > 0


def test_rounds_small_sampling_mode(harness):
    run = harness.ParityRun(synth.CONFIGS["small"])
    for r in range(4):
        run.round(p_m=0.6, check_draft=False, sample_seed=2024)
    print("sampling parity stats (small):", run.stats)
    assert run.stats["max_rel_logit"] <= 2e-2


def test_rounds_two_layer_head_two_taps(harness):
    """Multi-layer block head (Section 3.2): two head layers, the first fed by target layer 0 and the second by
    target layer 1.  Draft logits, tapped hidden states, per-layer head context K/V and the rounds against the
    oracle."""
    cfg = synth.CONFIGS["tiny"].replace(head_taps=(0, 1))
    run = harness.ParityRun(cfg)
    run.check_state()
    run.check_head_state()
    for r in range(6):
        run.round(p_m=(0.7 if r % 2 else None), check_draft=True)
    run.check_head_state()
    print("two-layer head parity stats:", run.stats)
    assert run.stats["max_rel_logit"] <= 2e-2


def test_rounds_small_three_layer_head(harness):
    """Three head layers tapping target layers 1, 4 and 7 of the 8-layer small configuration."""
    cfg = synth.CONFIGS["small"].replace(head_taps=(1, 4, 7))
    run = harness.ParityRun(cfg)
    run.check_head_state()
    for r in range(4):
        run.round(p_m=0.6, check_draft=(r < 2))
    run.check_head_state()
    print("three-layer head parity stats:", run.stats)
    assert run.stats["max_rel_logit"] <= 2e-2


def test_graph_replay_equals_plain_launches(harness):
    """One CUDA graph captured from a round serves every later round (all ragged quantities live in device memory):
    an engine replaying the graph and an engine making the four calls stay bit-identical over rounds with different
    trees and accept lengths."""
    from paper_2609_00355_b200.binding import Engine
    cfg = synth.CONFIGS["small"].replace(rounds=16)
    tw, hw = synth.make_weights(cfg, "cuda")
    img, ids = synth.make_context(cfg, "cuda")
    stream = torch.cuda.Stream()
    engines = []
    for use_stream in (None, stream):
        eng = Engine(cfg, tw, hw, batch=1, stream=use_stream)
        eng.prefill_context(0, img, ids)
        engines.append(eng)
    plain, graphed = engines
    L, k = cfg.L, cfg.topk
    cand_ids = torch.zeros(1, L, k, dtype=torch.int32, device="cuda")
    cand_lp = torch.from_numpy(synth.controlled_marginals(0.6, k, L))[None].cuda()
    rng = np.random.default_rng(5)

    def calls(eng):
        eng.glance_draft_block()
        eng.glance_build_tree(cand_ids, cand_lp)
        eng.glance_verify_tree()
        eng.glance_accept_commit()

    graph = None
    accepts = []
    for r in range(10):
        # plant the plain engine's true continuation so that accept lengths vary: look ahead with single-node trees
        snap = plain.snapshot_state()
        one = harness.TreeBuffers(1, cfg.tree_N, torch.device("cuda"))
        for i in range(cfg.tree_N):                 # every row sees itself only (tree_N <= 63 here)
            one.anc[0, i, 0] = 1 << i
        Y = []
        for _ in range(L):
            one.token[:, 0].copy_(plain.root)
            plain.glance_verify_tree(tree=one)
            plain.glance_accept_commit(tree=one)
            Y.append(int(plain.root[0]))
        plain.restore_state(snap)
        cand_ids.copy_(torch.from_numpy(synth.controlled_candidates(Y, 0.6, k, L, cfg.vocab, rng))[None])
        calls(plain)
        with torch.cuda.stream(stream):
            if r == 0:
                calls(graphed)                      # first round plain: sets up attributes and descriptors
            else:
                if graph is None:
                    snap_g = graphed.snapshot_state()
                    graph = graphed.capture(lambda: calls(graphed))
                    graphed.restore_state(snap_g)
                graph.replay()
        torch.cuda.synchronize()
        plain.check_device_status()
        graphed.check_device_status()
        accepts.append(int(plain.accept_len[0]))
        assert torch.equal(plain.seq_len, graphed.seq_len) and torch.equal(plain.root, graphed.root)
        assert torch.equal(plain.accept_len, graphed.accept_len) and torch.equal(plain.out_tokens, graphed.out_tokens)
        assert torch.equal(plain.topk_ids, graphed.topk_ids) and torch.equal(plain.topk_lp, graphed.topk_lp)
        P = int(plain.seq_len[0])
        for l in (0, cfg.n_layers - 1):
            Ka, Va = plain.gather_kv(0, l, P)
            Kb, Vb = graphed.gather_kv(0, l, P)
            assert torch.equal(Ka, Kb) and torch.equal(Va, Vb)
    assert len(set(accepts)) > 1, accepts


@pytest.mark.parametrize("block_B,topk,tree_N", [(2, 16, 2), (2, 1, 2), (16, 16, 128), (3, 2, 7), (16, 2, 33),
                                                 (4, 1, 8), (3, 2, 16)])
def test_rounds_extreme_block_topk_budget(harness, block_B, topk, tree_N):
    """Corners of the supported shapes: the shortest block (L = 1), the widest top-k, the smallest and the largest
    verify budget, budgets that the candidate trie cannot fill (n_nodes < N) and budgets that are not multiples of
    the GEMM row granularity."""
    cfg = synth.CONFIGS["tiny"].replace(block_B=block_B, topk=topk, tree_N=tree_N, rounds=8)
    run = harness.ParityRun(cfg)
    run.check_state()
    for r in range(3):
        run.round(p_m=(0.7 if r else None), check_draft=(r == 0))
    run.check_head_state()
    assert run.stats["max_rel_logit"] <= 2e-2


def test_rounds_batch2_sampling_two_layer_head(harness):
    """Everything at once on two ragged sequences: sampling walk, two-layer two-tap head, root-entropy log."""
    cfg = synth.CONFIGS["tiny"].replace(tree_N=16, block_B=6, topk=3, head_taps=(0, 1))
    run = harness.ParityRun(cfg, batch=2, ctx_lens=[(70, 19), (140, 33)])
    run.check_state()
    for r in range(5):
        run.round(p_m=(0.75 if r % 2 else None), check_draft=(r == 0), sample_seed=77)
    run.check_head_state()
    print("batch-2 sampling parity stats:", run.stats)
    assert run.stats["max_rel_logit"] <= 2e-2
