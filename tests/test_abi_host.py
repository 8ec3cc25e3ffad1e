"""Host-side checks of the C ABI that need no GPU: the library loads, exports every declared symbol,
sizes workspaces and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_2609_00355_b200 import build as glance_build
from paper_2609_00355_b200 import binding, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    glance_build.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "glance.h")).read()
    declared = set(re.findall(r"\b(glance_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert lib.glance_status_string(0) == b"ok"
    seen = {lib.glance_status_string(c) for c in range(-7, 1)}
    assert len(seen) == 8 and b"unknown status" not in seen
    assert lib.glance_status_string(-99) == b"unknown status"


def test_workspace_sizing_and_shape_validation(lib):
    sizes = {}
    for name in ("tiny", "small", "7b", "long"):
        cfg = synth.CONFIGS[name]
        cc = binding.make_config(cfg, 1, 200)
        sizes[name] = lib.glance_workspace_bytes(C.byref(cc))
        assert sizes[name] > 0
    assert sizes["tiny"] < sizes["small"] < sizes["7b"] <= sizes["long"]
    # 7B shape, 64 rows: residual + partial planes + fp32 logits stay far below 1 GB
    assert sizes["7b"] < 1 << 30
    bad = binding.make_config(synth.CONFIGS["tiny"].replace(head_dim=96), 1, 8)
    assert lib.glance_workspace_bytes(C.byref(bad)) == 0
    bad = binding.make_config(synth.CONFIGS["tiny"].replace(tree_N=256), 1, 8)
    assert lib.glance_workspace_bytes(C.byref(bad)) == 0
    bad = binding.make_config(synth.CONFIGS["tiny"].replace(block_B=17), 1, 8)
    assert lib.glance_workspace_bytes(C.byref(bad)) == 0
    bad = binding.make_config(synth.CONFIGS["tiny"].replace(page_size=32), 1, 8)
    assert lib.glance_workspace_bytes(C.byref(bad)) == 0
    # more candidates per offset than the vocabulary holds
    bad = binding.make_config(synth.CONFIGS["tiny"].replace(vocab=8, topk=9), 1, 8)
    assert lib.glance_workspace_bytes(C.byref(bad)) == 0
    # a one-row budget is plain decoding and is supported
    ok = binding.make_config(synth.CONFIGS["tiny"].replace(tree_N=1), 1, 8)
    assert lib.glance_workspace_bytes(C.byref(ok)) > 0
    # multi-layer head: taps must be distinct target layers; deeper heads need more workspace
    one = lib.glance_workspace_bytes(C.byref(binding.make_config(synth.CONFIGS["tiny"], 1, 8)))
    two = lib.glance_workspace_bytes(C.byref(binding.make_config(synth.CONFIGS["tiny"].replace(head_taps=(0, 1)), 1, 8)))
    assert two > one > 0
    for taps in ((0, 0), (0, 2), (-1, 1)):
        bad = binding.make_config(synth.CONFIGS["tiny"].replace(head_taps=taps), 1, 8)
        assert lib.glance_workspace_bytes(C.byref(bad)) == 0
    nine = binding.make_config(synth.CONFIGS["small"].replace(head_taps=(0, 1, 2, 3, 4, 5, 6, 7)), 1, 8)
    assert lib.glance_workspace_bytes(C.byref(nine)) > 0
    nine.head_layers = 9
    assert lib.glance_workspace_bytes(C.byref(nine)) == 0


def test_null_arguments_are_rejected_on_the_host(lib):
    cc = binding.make_config(synth.CONFIGS["tiny"], 1, 8)
    out = C.c_void_p()
    assert lib.glance_create(C.byref(cc), None, None, None, 0, None, C.byref(out)) == -1
    assert lib.glance_destroy(None) == -1
    assert lib.glance_poll_status(None, None) == -1
    assert lib.glance_build_tree(None, 1, None, None, None, None) == -1
    assert lib.glance_log_root_entropy(None, None) == -1
    assert lib.glance_verify_tree_sample(None, None, None, C.c_uint64(1), C.c_float(1.0), None, None, None) == -1
    assert lib.glance_launch_count(None) == 0


def test_no_oracle_import_in_product_path():
    """The product path never routes through the oracle (and has no CPU fallback)."""
    pkg = os.path.join(ROOT, "paper_2609_00355_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "glance_oracle" not in text and "import oracle" not in text and "from oracle" not in text, f
    otext = open(os.path.join(ROOT, "oracle", "glance_oracle.py")).read()
    assert "paper_2609_00355_b200" not in otext.replace("tests/", "")
