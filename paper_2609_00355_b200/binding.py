"""ctypes binding of libglance.so: the same entry points as include/glance.h, argument marshalling only.

PyTorch is used for device memory and streams; every step of the round runs in the library's CUDA
kernels.  There is no CPU fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libglance.so")

EXPORTS = [
    "glance_status_string", "glance_workspace_bytes", "glance_create", "glance_destroy", "glance_prefill",
    "glance_seq_truncate", "glance_draft_block", "glance_build_tree", "glance_verify_tree",
    "glance_verify_tree_sample", "glance_log_root_entropy",
    "glance_accept_commit", "glance_commit_forced", "glance_poll_status", "glance_launch_count",
    "glance_debug_attention", "glance_debug_gemm", "glance_profile_enable", "glance_profile_read",
    "glance_topk_static", "glance_debug_trace", "glance_debug_attention_terms", "glance_debug_stall_next_gemm",
]


class GlanceError(RuntimeError):
    pass


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_int32) for n in ("block_B", "topk", "tree_N", "page_size", "max_batch", "max_pages_per_seq")] + \
               [("head_layers", C.c_int32), ("head_taps", C.c_int32 * 8)]


class TargetWeights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("ln1", "wqkv", "wo", "ln2", "wgu", "wd")]


class HeadLayer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("ctx_norm", "ln1", "wqkv", "wo", "ln2", "wgu", "wd")]


class HeadWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("mask_embed", "ctx_norm", "ln1", "wqkv", "wo", "ln2", "wgu", "wd", "final_norm")] + \
               [("more", C.POINTER(HeadLayer))]


class Seqs(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_pages", C.c_int32), ("seq_len", C.c_void_p), ("root", C.c_void_p),
                ("page_table", C.c_void_p), ("kv_pool", C.c_void_p), ("head_kv_pool", C.c_void_p),
                ("feat", C.c_void_p), ("feat_count", C.c_void_p)]


class Tree(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("token", "parent", "depth", "rank", "score", "anc", "n_nodes")]


_lib = None


def load_library() -> C.CDLL:
    """Loads libglance.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise GlanceError(f"{LIB_PATH} not found: build it with `python -m paper_2609_00355_b200.build`")
    lib = C.CDLL(LIB_PATH)
    lib.glance_status_string.restype = C.c_char_p
    lib.glance_status_string.argtypes = [C.c_int32]
    lib.glance_workspace_bytes.restype = C.c_size_t
    lib.glance_workspace_bytes.argtypes = [C.POINTER(Config)]
    lib.glance_create.restype = C.c_int32
    lib.glance_create.argtypes = [C.POINTER(Config), C.POINTER(TargetWeights), C.POINTER(HeadWeights), C.c_void_p,
                                  C.c_size_t, C.c_void_p, C.POINTER(C.c_void_p)]
    lib.glance_destroy.restype = C.c_int32
    lib.glance_destroy.argtypes = [C.c_void_p]
    lib.glance_prefill.restype = C.c_int32
    lib.glance_prefill.argtypes = [C.c_void_p, C.POINTER(Seqs), C.c_int32, C.c_void_p, C.c_void_p, C.c_int32]
    lib.glance_seq_truncate.restype = C.c_int32
    lib.glance_seq_truncate.argtypes = [C.c_void_p, C.POINTER(Seqs), C.c_int32, C.c_int32, C.c_int32]
    lib.glance_draft_block.restype = C.c_int32
    lib.glance_draft_block.argtypes = [C.c_void_p, C.POINTER(Seqs), C.c_void_p, C.c_void_p, C.c_void_p]
    lib.glance_build_tree.restype = C.c_int32
    lib.glance_build_tree.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(Tree)]
    lib.glance_verify_tree.restype = C.c_int32
    lib.glance_verify_tree.argtypes = [C.c_void_p, C.POINTER(Seqs), C.POINTER(Tree), C.c_void_p, C.c_void_p, C.c_void_p]
    lib.glance_log_root_entropy.restype = C.c_int32
    lib.glance_log_root_entropy.argtypes = [C.c_void_p, C.c_void_p]
    lib.glance_verify_tree_sample.restype = C.c_int32
    lib.glance_verify_tree_sample.argtypes = [C.c_void_p, C.POINTER(Seqs), C.POINTER(Tree), C.c_uint64, C.c_float, C.c_void_p,
                                              C.c_void_p, C.c_void_p]
    lib.glance_accept_commit.restype = C.c_int32
    lib.glance_accept_commit.argtypes = [C.c_void_p, C.POINTER(Seqs), C.POINTER(Tree), C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.c_void_p]
    lib.glance_commit_forced.restype = C.c_int32
    lib.glance_commit_forced.argtypes = [C.c_void_p, C.POINTER(Seqs), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.glance_poll_status.restype = C.c_int32
    lib.glance_poll_status.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
    lib.glance_debug_attention.restype = C.c_int32
    lib.glance_debug_attention.argtypes = [C.c_void_p, C.POINTER(Seqs), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_int32, C.c_void_p, C.c_void_p]
    lib.glance_debug_gemm.restype = C.c_int32
    lib.glance_debug_gemm.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_int32, C.c_int32, C.c_int32, C.c_int32]
    lib.glance_profile_enable.restype = C.c_int32
    lib.glance_profile_enable.argtypes = [C.c_void_p, C.c_int32]
    lib.glance_profile_read.restype = C.c_int32
    lib.glance_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    lib.glance_debug_attention_terms.restype = C.c_int32
    lib.glance_debug_attention_terms.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
    lib.glance_debug_stall_next_gemm.restype = C.c_int32
    lib.glance_debug_stall_next_gemm.argtypes = [C.c_void_p, C.c_int32, C.c_uint64]
    lib.glance_debug_trace.restype = C.c_int32
    lib.glance_debug_trace.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
    lib.glance_topk_static.restype = C.c_int32
    lib.glance_topk_static.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                       C.c_void_p]
    lib.glance_launch_count.restype = C.c_int64
    lib.glance_launch_count.argtypes = [C.c_void_p]
    _lib = lib
    return lib


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise GlanceError(f"{what}: {load_library().glance_status_string(rc).decode()} ({rc})")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors only"
    return t.data_ptr()


def make_config(cfg, max_batch: int, max_pages_per_seq: int) -> Config:
    taps = tuple(getattr(cfg, "head_taps", ()) or ())
    return Config(cfg.n_layers, cfg.hidden, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.ffn, cfg.vocab,
                  cfg.rms_eps, cfg.rope_theta, cfg.block_B, cfg.topk, cfg.tree_N, cfg.page_size, max_batch,
                  max_pages_per_seq, len(taps), (C.c_int32 * 8)(*taps))


def glance_topk_static(logits: torch.Tensor, k: int, topk_ids: torch.Tensor, topk_lp: torch.Tensor) -> int:
    """Top-k + log-softmax of logits [batch][block_B][vocab] using the library's built-in scratch array.

    For callers that must not allocate device memory: no workspace, no context.  Returns the status code
    (0, or GLANCE_E_CAPACITY = -3 when the request exceeds the built-in 1 MiB scratch).  Runs on the
    current torch stream; calls that could overlap on the GPU must be serialised by the caller.
    """
    batch, B, V = logits.shape
    sp = torch.cuda.current_stream(logits.device).cuda_stream
    return int(load_library().glance_topk_static(_ptr(logits), batch, B, V, k, _ptr(topk_ids), _ptr(topk_lp), C.c_void_p(sp)))


class TreeBuffers:
    """Device arrays of a batch of candidate trees, laid out as glance_tree expects."""

    def __init__(self, batch: int, N: int, device):
        W = (N + 63) // 64
        i32 = dict(dtype=torch.int32, device=device)
        self.batch, self.N, self.W = batch, N, W
        self.token = torch.zeros(batch, N, **i32)
        self.parent = torch.full((batch, N), -1, **i32)
        self.depth = torch.zeros(batch, N, **i32)
        self.rank = torch.zeros(batch, N, **i32)
        self.score = torch.zeros(batch, N, dtype=torch.float32, device=device)
        self.anc = torch.zeros(batch, N, W, dtype=torch.int64, device=device)   # uint64 bit patterns
        self.n_nodes = torch.ones(batch, **i32)
        self.c = Tree(*[_ptr(t) for t in (self.token, self.parent, self.depth, self.rank, self.score, self.anc,
                                          self.n_nodes)])


class Engine:
    """Owns the device memory of one model + batch of sequences and forwards calls to the C ABI.

    weights: (target, head) dicts of CUDA bf16 tensors in the layout glance.h documents.
    """

    def __init__(self, cfg, target: dict, head: dict, batch: int = 1, max_len: Optional[int] = None,
                 stream: Optional[torch.cuda.Stream] = None):
        self.lib = load_library()
        self.cfg = cfg
        self.batch = batch
        self.device = target["embed"].device
        assert self.device.type == "cuda", "the library runs on a CUDA device only"
        self.stream = stream
        page = cfg.page_size
        max_len = max_len or (cfg.ctx + cfg.rounds * cfg.block_B + 2 * cfg.tree_N + page)
        self.pages_per_seq = (max_len + page - 1) // page
        self.n_pages = batch * self.pages_per_seq
        self.ccfg = make_config(cfg, batch, self.pages_per_seq)
        self._keep = [target, head]
        L = cfg.n_layers
        arr = lambda key: (C.c_void_p * L)(*[_ptr(lw[key]) for lw in target["layers"]])
        self._arrs = {k: arr(k) for k in ("ln1", "wqkv", "wo", "ln2", "wgu", "wd")}
        self.tw = TargetWeights(_ptr(target["embed"]), _ptr(target["lm_head"]), _ptr(target["final_norm"]),
                                *[C.cast(self._arrs[k], C.POINTER(C.c_void_p)) for k in ("ln1", "wqkv", "wo", "ln2", "wgu", "wd")])
        more = head.get("more", [])
        self._more = (HeadLayer * max(1, len(more)))(*[HeadLayer(*[_ptr(lw[k]) for k in ("ctx_norm", "ln1", "wqkv", "wo", "ln2", "wgu", "wd")])
                                                        for lw in more])
        self.hw = HeadWeights(*[_ptr(head[k]) for k in ("mask_embed", "ctx_norm", "ln1", "wqkv", "wo", "ln2", "wgu", "wd", "final_norm")],
                              C.cast(self._more, C.POINTER(HeadLayer)) if more else None)
        self.head_layers = 1 + len(more)
        assert self.head_layers == max(1, len(getattr(cfg, "head_taps", ()) or ())), "one head weight set per tap"
        nbytes = self.lib.glance_workspace_bytes(C.byref(self.ccfg))
        if nbytes == 0:
            raise GlanceError("configuration not supported by the library")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        dev = self.device
        i32 = dict(dtype=torch.int32, device=dev)
        self.seq_len = torch.zeros(batch, **i32)
        self.root = torch.zeros(batch, **i32)
        self.feat_count = torch.zeros(batch, **i32)
        T = self.head_layers
        # one slice per head layer (= per tapped target layer); .feat / .hidden / .head_kv_pool are slice 0
        self.feat_all = torch.zeros(T, batch, cfg.block_B, cfg.hidden, dtype=torch.bfloat16, device=dev)
        self.feat = self.feat_all[0]
        # page tables: a fixed random permutation of the pool so that logical and physical order differ
        g = torch.Generator().manual_seed(1234)
        perm = torch.randperm(self.n_pages, generator=g).to(torch.int32)
        self.page_table = perm.reshape(batch, self.pages_per_seq).contiguous().to(dev)
        kv_shape = (cfg.n_layers, self.n_pages, 2, cfg.n_kv_heads, page, cfg.head_dim)
        self.kv_pool = torch.zeros(kv_shape, dtype=torch.bfloat16, device=dev)
        self.head_kv_all = torch.zeros((T,) + kv_shape[1:], dtype=torch.bfloat16, device=dev)
        self.head_kv_pool = self.head_kv_all[0]
        self.seqs = Seqs(batch, self.n_pages, _ptr(self.seq_len), _ptr(self.root), _ptr(self.page_table),
                         _ptr(self.kv_pool), _ptr(self.head_kv_all), _ptr(self.feat_all), _ptr(self.feat_count))
        ctx = C.c_void_p()
        sp = stream.cuda_stream if stream is not None else torch.cuda.current_stream(dev).cuda_stream
        self._stream_ptr = sp
        _check(self.lib.glance_create(C.byref(self.ccfg), C.byref(self.tw), C.byref(self.hw), _ptr(self.workspace),
                                      nbytes, C.c_void_p(sp), C.byref(ctx)), "glance_create")
        self.ctx = ctx
        # default output buffers
        Lh, k, N, B = cfg.L, cfg.topk, cfg.tree_N, cfg.block_B
        self.topk_ids = torch.zeros(batch, Lh, k, **i32)
        self.topk_lp = torch.zeros(batch, Lh, k, dtype=torch.float32, device=dev)
        self.tree = TreeBuffers(batch, N, dev)
        self.argmax = torch.zeros(batch, N, **i32)
        self.hidden_all = torch.zeros(T, batch, N, cfg.hidden, dtype=torch.bfloat16, device=dev)
        self.hidden = self.hidden_all[0]
        self.accept_len = torch.zeros(batch, **i32)
        self.path = torch.zeros(batch, B, **i32)
        self.out_tokens = torch.zeros(batch, B, **i32)

    def close(self):
        if getattr(self, "ctx", None):
            self.lib.glance_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the C ABI, one method per entry point -------------------------------------------------
    def glance_prefill(self, seq: int, embeds: Optional[torch.Tensor] = None, ids: Optional[torch.Tensor] = None):
        count = embeds.shape[0] if embeds is not None else ids.shape[0]
        _check(self.lib.glance_prefill(self.ctx, C.byref(self.seqs), seq, _ptr(embeds), _ptr(ids), count), "glance_prefill")

    def glance_seq_truncate(self, seq: int, new_len: int, new_root: int):
        _check(self.lib.glance_seq_truncate(self.ctx, C.byref(self.seqs), seq, new_len, new_root), "glance_seq_truncate")

    def glance_draft_block(self, logits_dbg: Optional[torch.Tensor] = None):
        _check(self.lib.glance_draft_block(self.ctx, C.byref(self.seqs), _ptr(self.topk_ids), _ptr(self.topk_lp),
                                           _ptr(logits_dbg)), "glance_draft_block")

    def glance_build_tree(self, topk_ids: Optional[torch.Tensor] = None, topk_lp: Optional[torch.Tensor] = None,
                          root: Optional[torch.Tensor] = None, tree: Optional[TreeBuffers] = None):
        tree = tree or self.tree
        _check(self.lib.glance_build_tree(self.ctx, tree.batch, _ptr(self.root if root is None else root),
                                          _ptr(self.topk_ids if topk_ids is None else topk_ids),
                                          _ptr(self.topk_lp if topk_lp is None else topk_lp), C.byref(tree.c)),
               "glance_build_tree")

    def glance_verify_tree(self, tree: Optional[TreeBuffers] = None, logits_dbg: Optional[torch.Tensor] = None):
        tree = tree or self.tree
        _check(self.lib.glance_verify_tree(self.ctx, C.byref(self.seqs), C.byref(tree.c), _ptr(self.argmax),
                                           _ptr(self.hidden_all), _ptr(logits_dbg)), "glance_verify_tree")

    def glance_verify_tree_sample(self, seed: int, temperature: float = 1.0, tree: Optional[TreeBuffers] = None,
                                  logits_dbg: Optional[torch.Tensor] = None):
        """Sampling mode: self.argmax receives one draw per row instead of the arg-max."""
        tree = tree or self.tree
        _check(self.lib.glance_verify_tree_sample(self.ctx, C.byref(self.seqs), C.byref(tree.c), C.c_uint64(seed),
                                                  C.c_float(temperature), _ptr(self.argmax), _ptr(self.hidden_all),
                                                  _ptr(logits_dbg)), "glance_verify_tree_sample")

    def glance_log_root_entropy(self, entropy: Optional[torch.Tensor]):
        """entropy: float32 CUDA tensor [batch] that every later verify pass fills, or None to stop logging."""
        self._entropy_keep = entropy
        _check(self.lib.glance_log_root_entropy(self.ctx, _ptr(entropy)), "glance_log_root_entropy")

    def glance_accept_commit(self, tree: Optional[TreeBuffers] = None, argmax: Optional[torch.Tensor] = None):
        tree = tree or self.tree
        _check(self.lib.glance_accept_commit(self.ctx, C.byref(self.seqs), C.byref(tree.c),
                                             _ptr(self.argmax if argmax is None else argmax), _ptr(self.hidden_all),
                                             _ptr(self.accept_len), _ptr(self.path), _ptr(self.out_tokens)),
               "glance_accept_commit")

    def glance_commit_forced(self, path: torch.Tensor, path_len: torch.Tensor, new_root: torch.Tensor):
        _check(self.lib.glance_commit_forced(self.ctx, C.byref(self.seqs), _ptr(self.hidden_all), _ptr(path), _ptr(path_len),
                                             _ptr(new_root)), "glance_commit_forced")

    def glance_poll_status(self) -> int:
        v = C.c_int32(0)
        _check(self.lib.glance_poll_status(self.ctx, C.byref(v)), "glance_poll_status")
        return v.value

    def glance_debug_attention(self, layer: int, q: torch.Tensor, anc: Optional[torch.Tensor], T: int, out: torch.Tensor,
                               q_lo: Optional[torch.Tensor] = None, out_lo: Optional[torch.Tensor] = None):
        _check(self.lib.glance_debug_attention(self.ctx, C.byref(self.seqs), layer, _ptr(q), _ptr(q_lo), _ptr(anc), T,
                                               _ptr(out), _ptr(out_lo)), "glance_debug_attention")

    def glance_debug_gemm(self, mode: int, W, X, Y=None, act=None, argmax=None, S: int = 1):
        _check(self.lib.glance_debug_gemm(self.ctx, mode, _ptr(W), _ptr(X), _ptr(Y), _ptr(act), _ptr(argmax),
                                             W.shape[0], W.shape[1], X.shape[0], S), "glance_debug_gemm")

    def glance_debug_attention_terms(self, lo_skip: int, min_keys: int = 0):
        _check(self.lib.glance_debug_attention_terms(self.ctx, lo_skip, min_keys), "glance_debug_attention_terms")

    def glance_debug_stall_next_gemm(self, kstep: int, wait_limit_ns: int):
        _check(self.lib.glance_debug_stall_next_gemm(self.ctx, kstep, wait_limit_ns), "glance_debug_stall_next_gemm")

    def glance_debug_trace(self, buffer: Optional[torch.Tensor]):
        slots = 0 if buffer is None else buffer.numel() // 16
        _check(self.lib.glance_debug_trace(self.ctx, _ptr(buffer), slots), "glance_debug_trace")

    def glance_profile_enable(self, on: bool):
        _check(self.lib.glance_profile_enable(self.ctx, 1 if on else 0), "glance_profile_enable")

    def glance_profile_read(self):
        """Per kernel kind (gemm, attention, setup, control, other): (ms, algorithmic bytes, launches)."""
        ms, by, n = (C.c_double * 5)(), (C.c_double * 5)(), (C.c_int64 * 5)()
        _check(self.lib.glance_profile_read(self.ctx, ms, by, n), "glance_profile_read")
        names = ("gemm", "attention", "setup", "control", "other")
        return {names[i]: (ms[i], by[i], n[i]) for i in range(5)}

    def glance_launch_count(self) -> int:
        return int(self.lib.glance_launch_count(self.ctx))

    # ---- conveniences built only from the calls above ------------------------------------------
    def check_device_status(self):
        st = self.glance_poll_status()
        if st != 0:
            raise GlanceError(f"device status: {self.lib.glance_status_string(st).decode()} ({st})")

    def prefill_context(self, seq: int, image_embeds: torch.Tensor, text_ids: torch.Tensor):
        if image_embeds is not None and image_embeds.shape[0] > 0:
            self.glance_prefill(seq, embeds=image_embeds.contiguous())
        if text_ids is not None and text_ids.shape[0] > 0:
            self.glance_prefill(seq, ids=text_ids.contiguous())

    def round(self, use_draft_tree: bool = True):
        """One speculative round on the engine's own buffers (all four calls, stream-ordered)."""
        self.glance_draft_block()
        if use_draft_tree:
            self.glance_build_tree()
        self.glance_verify_tree()
        self.glance_accept_commit()

    def capture(self, fn):
        """Records the launches `fn()` makes on the engine's stream into a CUDA graph and returns the graph.

        The engine must have been created with its own (non-default) stream, and `fn` must already have run
        once (kernel attributes and TMA descriptors are set up on first use).  All ragged quantities (sequence
        lengths, accept lengths, page ids) are read from device memory by the kernels, so one graph serves
        every round.  Replay with graph.replay() while the engine's stream is current.
        """
        assert self.stream is not None, "create the Engine with its own stream to capture graphs"
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=self.stream):
            fn()
        return g

    def snapshot_state(self):
        return (self.seq_len.clone(), self.root.clone(), self.feat_all.clone(), self.feat_count.clone())

    def restore_state(self, snap):
        self.seq_len.copy_(snap[0]); self.root.copy_(snap[1]); self.feat_all.copy_(snap[2]); self.feat_count.copy_(snap[3])

    def gather_kv(self, seq: int, layer: int, length: int):
        """Logical K,V rows [length, Hkv, d] of one sequence and layer, read back through the page table (tests)."""
        return _gather(self.kv_pool[layer], self.page_table[seq], length, self.cfg.page_size)

    def gather_head_kv(self, seq: int, length: int, head_layer: int = 0):
        return _gather(self.head_kv_all[head_layer], self.page_table[seq], length, self.cfg.page_size)


def _gather(pool_layer: torch.Tensor, page_table: torch.Tensor, length: int, page: int):
    pos = torch.arange(length, device=pool_layer.device)
    pages = page_table.long()[pos // page]
    slots = pos % page
    K = pool_layer[pages, 0, :, slots, :]
    V = pool_layer[pages, 1, :, slots, :]
    return K, V
