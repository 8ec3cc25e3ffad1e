"""Stage-wise, teacher-forced comparison of the CUDA library with the CPU oracle (used by the gpu tests).

Because bf16 kernels and the fp32 oracle can disagree at near-ties, every round is compared stage by
stage on the same inputs, and the GPU is put back on the oracle's path whenever a near-tie sent it
elsewhere (the event is counted).  Tolerances:
  * logits, hidden states, log-probabilities, K/V rows: max-abs error <= 2e-2 x max|oracle tensor|
  * token ids (argmax, top-k): identical wherever the oracle's deciding margin exceeds 0.05
  * tree arrays, accepted path/length, emitted tokens, sequence state, compacted KV bytes: bit-exact
"""
import copy

import numpy as np
import torch

from oracle import glance_oracle as O
from paper_2609_00355_b200 import synth
from paper_2609_00355_b200.binding import Engine, TreeBuffers

REL_TOL = 2e-2
MARGIN = 0.05


def close(gpu: torch.Tensor, ref: torch.Tensor, what: str, scale=None):
    ref = ref.float()
    scale = float(ref.abs().max()) if scale is None else scale
    err = float((gpu.float().cpu() - ref).abs().max())
    assert err <= REL_TOL * scale, f"{what}: max-abs error {err:.4g} > {REL_TOL} x {scale:.4g}"
    return err / max(scale, 1e-30)


def tree_to_device(eng: Engine, trees, bufs: TreeBuffers = None) -> TreeBuffers:
    """Copies oracle Tree objects (one per sequence) into device buffers."""
    bufs = bufs or eng.tree
    for s, t in enumerate(trees):
        bufs.token[s] = torch.from_numpy(t.token)
        bufs.parent[s] = torch.from_numpy(t.parent)
        bufs.depth[s] = torch.from_numpy(t.depth)
        bufs.rank[s] = torch.from_numpy(t.rank)
        bufs.score[s] = torch.from_numpy(t.score)
        bufs.anc[s] = torch.from_numpy(t.anc.view(np.int64))
        bufs.n_nodes[s] = t.n_nodes
    return bufs


def tree_from_device(bufs: TreeBuffers, s: int) -> O.Tree:
    return O.Tree(bufs.token[s].cpu().numpy(), bufs.parent[s].cpu().numpy(), bufs.depth[s].cpu().numpy(),
                  bufs.rank[s].cpu().numpy(), bufs.score[s].cpu().numpy(),
                  bufs.anc[s].cpu().numpy().view(np.uint64), int(bufs.n_nodes[s]))


def assert_tree_bits(gpu: O.Tree, ref: O.Tree):
    assert gpu.n_nodes == ref.n_nodes
    for f in ("token", "parent", "depth", "rank"):
        assert np.array_equal(getattr(gpu, f), getattr(ref, f)), f
    assert np.array_equal(gpu.score.view(np.uint32), ref.score.view(np.uint32)), "score bits"
    assert np.array_equal(gpu.anc, ref.anc), "ancestor mask"


class ParityRun:
    def __init__(self, cfg, batch=1, ctx_lens=None, seed=0):
        self.cfg = cfg
        self.sh = O.Shape.of(cfg)
        self.batch = batch
        tw_b, hw_b = synth.make_weights(cfg, "cpu", seed)
        self.tw, self.hw = O.widen(tw_b), O.widen(hw_b)
        dev = torch.device("cuda:0")
        to_dev = lambda w: {k: ([{kk: vv.to(dev) for kk, vv in lw.items()} for lw in v] if isinstance(v, list) else v.to(dev))
                            for k, v in w.items()}
        self.eng = Engine(cfg, to_dev(tw_b), to_dev(hw_b), batch=batch)
        self.states = []
        self.stats = dict(rounds=0, forced=0, argmax_excused=0, topk_excused=0, max_rel_logit=0.0, accepted=0)
        ctx_lens = ctx_lens or [(cfg.n_img, cfg.n_txt)] * batch
        cap = max(a + b for a, b in ctx_lens) + cfg.rounds * cfg.block_B + 2 * cfg.tree_N + 64
        for s, (n_img, n_txt) in enumerate(ctx_lens):
            img, ids = synth.make_context(cfg, "cpu", seed=1 + s, n_img=n_img, n_txt=n_txt)
            ctx = O.context_embeddings(self.tw, img, ids.numpy())
            self.states.append(O.prefill(self.sh, self.tw, self.hw, ctx, cap))
            self.eng.prefill_context(s, img.to(dev), ids.to(dev))
        self.eng.check_device_status()
        # the root after prefill is an argmax: identical unless the oracle's margin is a near-tie
        for s, st in enumerate(self.states):
            g_root = int(self.eng.root[s])
            if g_root != st.root:
                lg = O.rmsnorm(st.feat[st.P - 1:st.P], self.tw["final_norm"], self.sh.rms_eps) @ self.tw["lm_head"].T
                top2 = torch.topk(lg[0], 2).values
                assert float(top2[0] - top2[1]) <= MARGIN, "prefill root differs at a clear margin"
                self.eng.glance_seq_truncate(s, st.P, st.root)
                self.stats["forced"] += 1
        self.rng = np.random.default_rng(7)
        # round log: root entropy of every verify pass
        self.entropy = torch.zeros(batch, dtype=torch.float32, device=dev)
        self.eng.glance_log_root_entropy(self.entropy)

    # ---- state comparison -------------------------------------------------------------------
    def check_state(self, check_root=True):
        eng = self.eng
        P = eng.seq_len.cpu().tolist()
        for s, st in enumerate(self.states):
            assert P[s] == st.P, f"seq_len[{s}]"
            if check_root:
                assert int(eng.root[s]) == st.root, f"root[{s}]"
            for l in range(self.cfg.n_layers):
                K, V = eng.gather_kv(s, l, st.P)
                close(K, st.K[l][:st.P], f"K layer {l} seq {s}")
                close(V, st.V[l][:st.P], f"V layer {l} seq {s}")

    def check_head_state(self):
        # head context K/V of positions already folded in (everything except the pending feat rows)
        for s, st in enumerate(self.states):
            n = st.P - int(self.eng.feat_count[s])
            if n > 0:
                for i in range(self.eng.head_layers):
                    K, V = self.eng.gather_head_kv(s, n, i)
                    close(K, (st.hK if i == 0 else st.hK_more[i - 1])[:n], f"head layer {i} K seq {s}")
                    close(V, (st.hV if i == 0 else st.hV_more[i - 1])[:n], f"head layer {i} V seq {s}")

    # ---- oracle look-ahead: the greedy continuation after the pending root -------------------
    def oracle_continuation(self, s: int, n: int, sample_seed=None):
        st = copy.deepcopy(self.states[s])
        Y = []
        for _ in range(n):
            if sample_seed is None:
                info = O.spec_round(self.sh, self.tw, self.hw, st, self.cfg.block_B, self.cfg.topk, 1,
                                    tree=O.chain_tree(st.root, [], 1))
            else:
                info = O.spec_round_sampled(self.sh, self.tw, self.hw, st, self.cfg.block_B, self.cfg.topk, 1,
                                            sample_seed, tree=O.chain_tree(st.root, [], 1))
            Y.append(info["new_root"])
        return Y

    # ---- one teacher-forced round -------------------------------------------------------------
    def round(self, p_m=None, check_draft=True, sample_seed=None):
        """sample_seed: run the round in sampling mode (temperature 1) with this seed instead of greedily."""
        cfg, eng, sh = self.cfg, self.eng, self.sh
        B, k, N, L, V = cfg.block_B, cfg.topk, cfg.tree_N, cfg.L, cfg.vocab
        dev = eng.device
        # (1) draft block: logits, top-k ids, log-probabilities
        dlog = torch.zeros(self.batch, B, V, dtype=torch.float32, device=dev)
        eng.glance_draft_block(logits_dbg=dlog)
        ids_g, lp_g = eng.topk_ids.cpu().numpy(), eng.topk_lp.cpu().numpy()
        if check_draft:
            for s, st in enumerate(self.states):
                ol = O.draft_block(sh, self.tw, self.hw, st, B)
                scale = float(ol[1:].abs().max())
                self.stats["max_rel_logit"] = max(self.stats["max_rel_logit"], close(dlog[s, 1:], ol[1:], "draft logits", scale))
                oid, olp = O.topk_logprobs(ol, k)
                srt = torch.sort(ol, dim=-1, descending=True).values.numpy()
                for j in range(L):
                    for r in range(k):
                        gap_hi = srt[j + 1][r - 1] - srt[j + 1][r] if r > 0 else np.inf
                        gap_lo = srt[j + 1][r] - srt[j + 1][r + 1]
                        if gap_hi > MARGIN and gap_lo > MARGIN:
                            assert ids_g[s, j, r] == oid[j, r], f"top-k id offset {j + 1} rank {r}"
                            assert abs(lp_g[s, j, r] - olp[j, r]) <= REL_TOL * scale
                        else:
                            self.stats["topk_excused"] += 1
                # the library's own (ids, lp) must be self-consistent: lp = its logit - its lse
                lse = torch.logsumexp(dlog[s, 1:].double(), dim=-1).cpu()
                own = torch.gather(dlog[s, 1:].cpu().double(), 1, torch.from_numpy(ids_g[s]).long()) - lse[:, None]
                assert float((own - torch.from_numpy(lp_g[s]).double()).abs().max()) < 1e-3
                assert np.all(np.diff(lp_g[s], axis=1) <= 0)
        # (2) tree: either from the library's own draft output or from controlled-match candidates
        Ys = None
        if p_m is not None:
            Ys = [self.oracle_continuation(s, L + 1, sample_seed) for s in range(self.batch)]
            lp_c = synth.controlled_marginals(p_m, k, L)
            ids_in = np.stack([synth.controlled_candidates(Ys[s][:L], p_m, k, L, V, self.rng) for s in range(self.batch)])
            lp_in = np.stack([lp_c] * self.batch)
            eng.glance_build_tree(torch.from_numpy(ids_in).to(dev), torch.from_numpy(lp_in).to(dev))
        else:
            ids_in, lp_in = ids_g, lp_g
            eng.glance_build_tree()
        roots = eng.root.cpu().tolist()
        trees = []
        for s in range(self.batch):
            ref = O.build_tree(roots[s], ids_in[s], lp_in[s], N)
            assert_tree_bits(tree_from_device(eng.tree, s), ref)
            trees.append(ref)
        # (3) verify
        vlog = torch.zeros(self.batch, N, V, dtype=torch.float32, device=dev)
        pool_before = eng.kv_pool.clone()
        state_before = eng.snapshot_state()
        if sample_seed is None:
            eng.glance_verify_tree(logits_dbg=vlog)
        else:
            eng.glance_verify_tree_sample(sample_seed, 1.0, logits_dbg=vlog)
        am_g = eng.argmax.cpu().numpy()
        ent_g = self.entropy.cpu().numpy()
        infos = []
        for s, st in enumerate(self.states):
            assert roots[s] == st.root
            ol, oh = O.verify_tree(sh, self.tw, st, trees[s])
            n = trees[s].n_nodes
            scale = float(ol[:n].abs().max())
            self.stats["max_rel_logit"] = max(self.stats["max_rel_logit"], close(vlog[s, :n], ol[:n], "verify logits", scale))
            for i, oh_i in enumerate([oh] if oh.dim() == 2 else list(oh)):       # one slice per tapped layer
                close(eng.hidden_all[i, s, :n], oh_i[:n], f"verify hidden, tap {i}")
            # root entropy (Section 4): exact on the library's own logits, within the logit tolerance of the oracle's
            own_H = O.root_entropy(vlog[s, 0].cpu())
            assert abs(float(ent_g[s]) - own_H) <= 1e-3 * max(1.0, own_H), f"root entropy {ent_g[s]} vs {own_H} on own logits"
            assert abs(float(ent_g[s]) - O.root_entropy(ol[0])) <= 4 * REL_TOL * scale, "root entropy against the oracle"
            if sample_seed is None:
                oam = O.argmax_lowest(ol)
                top2 = torch.topk(ol, 2, dim=-1).values
                margin = (top2[:, 0] - top2[:, 1]).numpy()
            else:
                # one draw per row: arg-max of the row perturbed by the noise field of the predicted position
                positions = [st.P + int(d) + 1 for d in trees[s].depth]
                oam, margin = O.sample_rows(ol, positions, sample_seed)
            for i in range(n):
                if margin[i] > MARGIN:
                    assert am_g[s, i] == oam[i], f"decision row {i} (margin {margin[i]:.3f})"
                elif am_g[s, i] != oam[i]:
                    self.stats["argmax_excused"] += 1
            if sample_seed is None:
                # the library's argmax is the argmax of its own fp32 logits, ties to the lowest id
                assert np.array_equal(am_g[s], O.argmax_lowest(vlog[s].cpu()))
            else:
                # the library's draws are the arg-max of its own logits plus the same noise field (the two sides
                # evaluate the logarithms of the Gumbel transform independently: near-ties are exempt)
                own, own_margin = O.sample_rows(vlog[s].cpu(), positions, sample_seed)
                for i in range(n):
                    assert am_g[s, i] == own[i] or own_margin[i] < 1e-3, f"draw row {i} is not the perturbed arg-max"
            infos.append((ol, oh, oam))
        # tree K/V rows written at P + i
        for s, st in enumerate(self.states):
            for l in range(cfg.n_layers):
                K, V_ = eng.gather_kv(s, l, st.P + N)
                close(K[st.P:], st.K[l][st.P:st.P + N], f"tree K layer {l}", float(st.K[l][:st.P + N].abs().max()))
                close(V_[st.P:], st.V[l][st.P:st.P + N], f"tree V layer {l}", float(st.V[l][:st.P + N].abs().max()))
        # (4) walk + commit on the library's own argmax, against the oracle walk on the same array
        pool_verified = eng.kv_pool.clone()
        eng.glance_accept_commit()
        eng.check_device_status()
        a_g = eng.accept_len.cpu().numpy()
        path_g, out_g = eng.path.cpu().numpy(), eng.out_tokens.cpu().numpy()
        need_force = False
        for s, st in enumerate(self.states):
            a, path, out, new_root = O.walk(trees[s], am_g[s])
            assert a_g[s] == a and list(path_g[s, :a + 1]) == path and list(out_g[s, :a]) == out
            assert out_g[s, a] == new_root and int(eng.root[s]) == new_root
            assert int(eng.seq_len[s]) == st.P + a + 1 and int(eng.feat_count[s]) == a + 1
            self._check_compaction(s, st.P, path, pool_verified)
            for i in range(eng.head_layers):
                assert torch.equal(eng.feat_all[i, s, :a + 1], eng.hidden_all[i, s, torch.tensor(path, device=dev)])
            oa, opath, oout, oroot = O.walk(trees[s], infos[s][2])
            if (a, path, new_root) != (oa, opath, oroot):
                need_force = True
            if Ys is not None:
                assert oa == O.accepted_length_bruteforce(trees[s], Ys[s])
        # (5) the oracle commits its own path; a GPU that left it is put back with glance_commit_forced
        if need_force:
            self.stats["forced"] += 1
            eng.kv_pool.copy_(pool_verified)
            eng.restore_state(state_before)
            paths = torch.full((self.batch, B), -1, dtype=torch.int32)
            lens = torch.zeros(self.batch, dtype=torch.int32)
            nroots = torch.zeros(self.batch, dtype=torch.int32)
            for s in range(self.batch):
                oa, opath, oout, oroot = O.walk(trees[s], infos[s][2])
                paths[s, :oa + 1] = torch.tensor(opath, dtype=torch.int32)
                lens[s] = oa + 1
                nroots[s] = oroot
            eng.glance_commit_forced(paths.to(dev), lens.to(dev), nroots.to(dev))
            eng.check_device_status()
            for s, st in enumerate(self.states):
                oa, opath, _, _ = O.walk(trees[s], infos[s][2])
                self._check_compaction(s, st.P, opath, pool_verified)
        for s, st in enumerate(self.states):
            ol, oh, oam = infos[s]
            oa, opath, oout, oroot = O.walk(trees[s], oam)
            O.commit(sh, self.hw, st, opath, oh, oout, oroot)
            self.stats["accepted"] += oa
        self.stats["rounds"] += 1
        del pool_before
        self.check_state()

    def _check_compaction(self, s, P, path, pool_verified):
        """Rows P..P+a after the commit are byte-identical to rows P+path[d] before it; rows < P untouched."""
        eng = self.eng
        page = self.cfg.page_size
        pt = eng.page_table[s].long()
        for d, v in enumerate(path):
            dst, src = P + d, P + v
            now = eng.kv_pool[:, pt[dst // page], :, :, dst % page, :]
            was = pool_verified[:, pt[src // page], :, :, src % page, :]
            assert torch.equal(now, was), f"compacted row {d}"
        pos = torch.arange(P, device=eng.device)
        assert torch.equal(eng.kv_pool[:, pt[pos // page], :, :, pos % page, :],
                           pool_verified[:, pt[pos // page], :, :, pos % page, :]), "committed rows changed"
