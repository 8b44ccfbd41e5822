"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every symbol the header declares, sizes workspaces and rejects bad arguments
before touching a device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def rv():
    from paper_2512_20920_b200 import build
    build.build()
    import paper_2512_20920_b200 as rv
    return rv


def _declared_functions():
    inc = os.path.join(ROOT, "include")
    names = set()
    for f in sorted(os.listdir(inc)):
        if not f.endswith(".h"):
            continue
        text = open(os.path.join(inc, f)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(revffn_\w+)\s*\(", text))
    return sorted(names)


def test_header_symbols_are_exported(rv):
    names = _declared_functions()
    assert {"revffn_moe_forward", "revffn_moe_inverse", "revffn_moe_backward", "revffn_moe_workspace_size",
            "revffn_moe_status", "revffn_strerror", "revffn_attn_forward", "revffn_attn_inverse",
            "revffn_attn_backward", "revffn_attn_workspace_size", "revffn_attn_status"} <= set(names)
    for n in names:
        assert hasattr(rv.lib, n), n


def _desc(rv, **kw):
    base = dict(tokens=8192, d_model=2048, n_experts=60, top_k=4, d_expert=1408, d_shared=5632,
                weight_dtype=rv.BF16, norm_kind=rv.NORM_RMS, norm_eps=1e-6, ld_stream=1024, flags=0)
    base.update(kw)
    return rv.Desc(**base)


def test_workspace_size_c1(rv):
    fwd, bwd = rv.revffn_moe_workspace_size(_desc(rv))
    rows_pad = ((8192 * 4 + 60 * 127 + 127) // 128) * 128
    # the permuted activations alone: Up, H, O in bf16
    assert fwd > rows_pad * (2048 + 1408 + 2048) * 2
    assert bwd > fwd
    assert bwd < 4 * 2**30
    f0, b0 = rv.revffn_moe_workspace_size(_desc(rv, tokens=0))
    assert 0 < f0 < fwd


@pytest.mark.parametrize("kw", [dict(d_model=2047), dict(top_k=0), dict(top_k=9), dict(n_experts=3),
                                dict(n_experts=300), dict(d_expert=1400), dict(d_shared=100), dict(tokens=-1),
                                dict(weight_dtype=7), dict(norm_kind=5)])
def test_bad_descriptors_are_rejected(rv, kw):
    with pytest.raises(rv.RevffnError) as e:
        rv.revffn_moe_workspace_size(_desc(rv, **kw))
    assert e.value.code == -2


def test_bad_stream_stride_is_rejected(rv):
    with pytest.raises(rv.RevffnError) as e:
        rv.revffn_moe_workspace_size(_desc(rv, ld_stream=1000))
    assert e.value.code == -3


def test_null_and_misaligned_pointers_are_rejected_before_any_launch(rv):
    d = _desc(rv)
    w = rv.Weights()
    code = rv.lib.revffn_moe_forward(C.byref(d), C.byref(w), 0x1000, 0x1000, 0x1000, None, 0x1000, 1 << 40, None)
    assert code == -1          # weights missing
    fake = {n: 0x10000 for n, _ in rv.Weights._fields_}
    w = rv.Weights(**fake)
    code = rv.lib.revffn_moe_forward(C.byref(d), C.byref(w), 0x1000, 0x1000, 0x1000, None, None, 1 << 40, None)
    assert code == -1          # workspace missing
    code = rv.lib.revffn_moe_forward(C.byref(d), C.byref(w), 0x1004, 0x1000, 0x1000, None, 0x1000, 1 << 40, None)
    assert code == -3          # misaligned stream
    code = rv.lib.revffn_moe_forward(C.byref(d), C.byref(w), 0x1000, 0x1000, 0x1000, None, 0x1000, 1024, None)
    assert code == -4          # workspace too small
    code = rv.lib.revffn_moe_backward(C.byref(d), C.byref(w), 0x1000, 0x1000, 0x1000, None, None, 0x1000, 1 << 40, None)
    assert code == -1          # grads struct missing


def test_strerror(rv):
    assert rv.revffn_strerror(0) == "ok"
    assert "workspace" in rv.revffn_strerror(-4)
    assert rv.revffn_strerror(-1234) == "unknown error"


def test_ws_lookup(rv):
    from paper_2512_20920_b200 import binding
    d = _desc(rv)
    off_u, n_u = binding.ws_lookup(d, "u")
    assert n_u == 8192 * 2048 * 2 and off_u % 256 == 0
    with pytest.raises(rv.RevffnError):
        binding.ws_lookup(d, "no_such_buffer")


def _attn_desc(rv, **kw):
    base = dict(batch=4, seq_len=2048, d_model=2048, n_heads=16, n_kv_heads=16, weight_dtype=rv.BF16, norm_eps=1e-6,
                rope_theta=1e6, ld_stream=1024, flags=0)
    base.update(kw)
    return rv.AttnDesc(**base)


def test_attention_workspace_size_and_bad_descriptors(rv):
    fwd, bwd = rv.revffn_attn_workspace_size(_attn_desc(rv))
    rows = 4 * 16 * 2048
    assert fwd > rows * 2048 * (4 + 2)          # the score matrix in fp32 and P in bf16
    assert fwd < bwd < 8 * 2**30
    f2, _ = rv.revffn_attn_workspace_size(_attn_desc(rv, seq_len=2000))     # rows padded to 128 per head
    assert f2 > rv.revffn_attn_workspace_size(_attn_desc(rv, seq_len=1920))[0]
    for kw in (dict(d_model=2047), dict(n_heads=15), dict(n_kv_heads=3), dict(seq_len=0), dict(batch=-1),
               dict(n_heads=32), dict(weight_dtype=5), dict(rope_theta=0.0)):
        with pytest.raises(rv.RevffnError) as e:
            rv.revffn_attn_workspace_size(_attn_desc(rv, **kw))
        assert e.value.code == -2, kw
    with pytest.raises(rv.RevffnError) as e:
        rv.revffn_attn_workspace_size(_attn_desc(rv, flags=rv.FLAG_SAVE_ACTIVATIONS))
    assert e.value.code == -8


def test_block_workspace_is_the_larger_branch_plus_one_stream(rv):
    a = _attn_desc(rv)
    m = _desc(rv)
    d = rv.BlockDesc(a, m, 1)
    fwd, bwd = rv.revffn_block_workspace_size(d)
    af, ab = rv.revffn_attn_workspace_size(a)
    mf, mb = rv.revffn_moe_workspace_size(m)
    stream = 8192 * 1024 * 4
    assert max(af, mf) + stream <= fwd <= max(af, mf) + stream + 4096
    assert max(ab, mb) + stream <= bwd <= max(ab, mb) + stream + 4096
    # the two halves of a block must describe the same tokens
    for bad in (rv.BlockDesc(_attn_desc(rv, seq_len=1024), m, 1), rv.BlockDesc(_attn_desc(rv, d_model=1024, n_heads=8, n_kv_heads=8, ld_stream=512), m, 1),
                rv.BlockDesc(a, _desc(rv, ld_stream=2048), 1), rv.BlockDesc(a, m, -1)):
        with pytest.raises(rv.RevffnError) as e:
            rv.revffn_block_workspace_size(bad)
        assert e.value.code == -2


def test_schedule_stages_select_the_trainable_weights(rv):
    a1, m1 = rv.trainable_names(1)
    assert set(a1) == {"w_up", "w_down"} and set(m1) == {"w_up", "w_down"}          # adapters only
    a2, m2 = rv.trainable_names(2)
    assert "w_q" in a2 and "norm_gamma" in a2 and "w_gate" in m2 and "ws_down" in m2
    assert "w_router" not in m2 and "b_router" not in m2                            # the router stays frozen
    with pytest.raises(ValueError):
        rv.trainable_names(3)
