"""The C-ABI library loads and exports every symbol the public header declares; host-side argument
checks work without a GPU (no compute call is made here)."""
import ctypes
import os
import re

import pytest
import torch

from paper_2503_00540_b200 import rekv

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(rekv_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    lib = rekv.lib()
    declared = _declared()
    assert {"rekv_create", "rekv_append_frame", "rekv_retrieve", "rekv_gather", "rekv_attend"} <= declared
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in include/ but not exported"
    assert declared == set(rekv.EXPORTS) | {n for n in declared if n not in rekv.EXPORTS}
    missing_binding = declared - set(rekv.EXPORTS)
    assert not missing_binding, f"no Python binding for {missing_binding}"


def test_config_struct_matches_header_layout():
    assert ctypes.sizeof(rekv.rekv_config) == 17 * 4
    assert ctypes.sizeof(rekv.rekv_stats_t) == 7 * 8 + 2 * 4 + 4 * 8  # seven counters, two ints, four stage timings


def test_create_rejects_bad_shapes_before_touching_a_device():
    for kwargs, frag in [
        (dict(head_dim=64), "head_dim"),
        (dict(n_q_heads=7), "head counts"),
        (dict(tokens_per_frame=0), "tokens_per_frame"),
        (dict(tokens_per_frame=1025), "tokens_per_frame"),
        (dict(block_frames=0), "block_frames"),
        (dict(block_frames=3, max_topk=64), "multiple of block_frames"),
        (dict(hbm_tail_frames=2, window_frames=4), "window_frames"),
        (dict(max_questions=65), "max_questions"),
        (dict(rope_theta=0.5), "rope_theta"),
        (dict(max_self_tokens=-1), "max_self_tokens"),
        (dict(ext_embed_dim=1150), "ext_embed_dim"),
    ]:
        base = dict(n_layers=1, n_q_heads=8, n_kv_heads=2, head_dim=128, tokens_per_frame=16, max_frames=8,
                    window_frames=2)
        base.update(kwargs)
        with pytest.raises(rekv.RekvError) as e:
            rekv.ReKV(**base)
        assert e.value.code == rekv.ERR_ARG and frag in str(e.value)


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device failure")
def test_create_fails_loudly_without_a_device():
    with pytest.raises(rekv.RekvError) as e:
        rekv.ReKV(1, 8, 2, 128, 16, 8, 2)
    assert e.value.code == rekv.ERR_CUDA and "no CPU path" in str(e.value)


def test_null_context_calls_return_arg_error():
    lib = rekv.lib()
    assert lib.rekv_destroy(None) == rekv.ERR_ARG
    assert lib.rekv_append_frame(None, None, None, None) == rekv.ERR_ARG
    assert lib.rekv_attend(None, None, None, 1, None, None) == rekv.ERR_ARG


def test_geometry_call_rejects_a_null_context():
    assert rekv.lib().rekv_geometry(None, 10, 4, None, None, None) == rekv.ERR_ARG
