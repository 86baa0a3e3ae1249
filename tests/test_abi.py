"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import os
import re

import paper_2609_39361_b200 as lamp
from paper_2609_39361_b200 import build as lamp_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lamp_build.build()
    L = lamp.library()
    header = open(os.path.join(ROOT, "include", "lamp_attn.h")).read()
    declared = set(re.findall(r"\b(lamp_attn_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(L, name), name
    assert set(lamp.binding.EXPORTS) == declared


def test_host_only_calls_work_without_a_device():
    p = lamp.lamp_attn_default_params()
    assert p.threshold == 0.5 and p.delta == 2.0 ** -8 and p.causal == 1
    p.batch, p.heads_q, p.heads_kv, p.seqlen, p.head_dim = 2, 8, 4, 256, 128
    lamp.lamp_attn_contiguous_strides(p)
    assert list(p.q_strides) == [8 * 256 * 128, 256 * 128, 128]
    assert list(p.k_strides) == [4 * 256 * 128, 256 * 128, 128]
    assert lamp.lamp_attn_workspace_bytes(p) == 0
    # staging space of the host-memory call: Q, K, V, O (bf16), lse (fp32), flag mask (one byte per 32 x 64 tile)
    head = 256 * 128 * 2
    assert lamp.lamp_attn_host_workspace_bytes(p) == 16 * head + 2 * 8 * head + 16 * head + 16 * 256 * 4 + 16 * 8 * 4
    p.seqlen, p.flags, p.group_rows = 200, lamp.LAMP_OUT_FP32, 16         # ragged length, fp32 out, 16-row groups
    al = lambda x: (x + 255) // 256 * 256
    assert lamp.lamp_attn_host_workspace_bytes(p) == (al(16 * 200 * 128 * 2) + 2 * al(8 * 200 * 128 * 2) + al(16 * 200 * 128 * 4)
                                                      + al(16 * 200 * 4) + al(16 * 13 * 4))
    p.head_dim = 64
    assert lamp.lamp_attn_host_workspace_bytes(p) == 0                    # not a supported problem
    assert lamp.lamp_attn_strerror(0) == "ok" and "shape" in lamp.lamp_attn_strerror(-2)


def test_struct_layout_matches_header():
    import ctypes as C
    assert C.sizeof(lamp.LampAttnParams) == 184
    assert C.sizeof(lamp.LampAttnStats) == 168
