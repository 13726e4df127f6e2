"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the header
declares, sizes workspaces, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2506_16640_b200 import build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    lib_build.build()
    from paper_2506_16640_b200 import binding
    return binding.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "entmax_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(entmax_attn_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert {"entmax_attn_fwd", "entmax_attn_bwd", "entmax_attn_workspace_bytes", "entmax_attn_strerror"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def _params(**kw):
    from paper_2506_16640_b200.binding import Params
    base = dict(batch=1, heads=2, seq=128, head_dim=64, dtype=1, causal=1, n_mode=0, alpha=1.5, sm_scale=0.0,
                stride_b=0, stride_h=0, stride_n=0)
    base.update(kw)
    return Params(**base)


def test_workspace_bytes_and_layout(lib):
    from paper_2506_16640_b200.binding import WsLayout
    p = _params()
    fwd = lib.entmax_attn_workspace_bytes(ctypes.byref(p), 0)
    bwd = lib.entmax_attn_workspace_bytes(ctypes.byref(p), 1)
    rows = 1 * 2 * 128
    assert fwd >= rows * 256 * 8 and bwd >= fwd + 2 * rows * 64 * 4
    lay = WsLayout()
    assert lib.entmax_attn_workspace_layout(ctypes.byref(p), ctypes.byref(lay)) == 0
    assert lay.capacity == 256 and lay.entries_offset % 256 == 0 and lay.row_count_offset % 256 == 0
    big = _params(batch=1, heads=16, seq=32768, head_dim=128, dtype=0)
    assert lib.entmax_attn_workspace_bytes(ctypes.byref(big), 0) < 2 << 30
    for bad in [_params(head_dim=96), _params(seq=0), _params(alpha=1.0), _params(alpha=64.5), _params(dtype=7),
                _params(alpha=float("nan")), _params(stride_b=8, stride_h=8, stride_n=4)]:
        assert lib.entmax_attn_workspace_bytes(ctypes.byref(bad), 0) == 0


def test_rejections_happen_before_any_device_work(lib):
    p = _params()
    nul = ctypes.c_void_p(0)
    fake = ctypes.c_void_p(4096)      # aligned, never dereferenced: rejected earlier
    odd = ctypes.c_void_p(4100)
    rc = lib.entmax_attn_fwd(ctypes.byref(p), nul, fake, fake, None, None, None, fake, fake, fake, 1 << 30, None, None)
    assert rc == -6
    rc = lib.entmax_attn_fwd(ctypes.byref(p), fake, fake, fake, fake, None, None, fake, fake, fake, 1 << 30, None, None)
    assert rc == -6                   # beta without gamma/delta
    rc = lib.entmax_attn_fwd(ctypes.byref(p), odd, fake, fake, None, None, None, fake, fake, fake, 1 << 30, None, None)
    assert rc == -4
    rc = lib.entmax_attn_fwd(ctypes.byref(p), fake, fake, fake, None, None, None, fake, fake, fake, 16, None, None)
    assert rc == -5                   # workspace too small
    rc = lib.entmax_attn_fwd(ctypes.byref(p), fake, fake, fake, None, None, None, fake, fake, nul, 1 << 30, None, None)
    assert rc == -5
    bad = _params(alpha=0.5)
    rc = lib.entmax_attn_bwd(ctypes.byref(bad), fake, fake, fake, None, None, None, fake, fake, fake, fake, fake, fake,
                             1 << 30, None, None)
    assert rc == -2
    rc = lib.entmax_attn_bwd(ctypes.byref(_params(head_dim=32)), fake, fake, fake, None, None, None, fake, fake, fake,
                             fake, fake, fake, 1 << 30, None, None)
    assert rc == -1
    rc = lib.entmax_attn_scores_debug(ctypes.byref(p), fake, fake, 0, fake, fake, 1 << 30, None, None)
    assert rc == -3                   # fp32 params: the score engine is bf16 only
    for code in range(-8, 1):
        assert len(lib.entmax_attn_strerror(code)) > 0
    assert lib.entmax_attn_version() >= 100


def test_static_entry_point_size_limit_is_what_the_header_says(lib):
    # return codes only, no device work: the size check comes before the pointer checks, so a problem that
    # fits is rejected for its NULL tensors (-6) and one that does not fit for its size (-9).
    # limit: round_up(heads*seq, 32) + 64*round_up(seq, 32) floats <= 8 MiB; 16 heads: seq 26208 fits, 26209 does not
    nul = ctypes.c_void_p(0)
    call = lambda p: lib.entmax_attn_fwd_static(ctypes.byref(p), nul, nul, nul, None, None, None, nul, nul, None, None)
    assert call(_params(heads=16, seq=26208, dtype=0)) == -6
    assert call(_params(heads=16, seq=26209, dtype=0)) == -9
    assert call(_params(heads=16, seq=26214, dtype=0)) == -9
    assert call(_params(heads=1, seq=32256, dtype=0)) == -6       # 32256 + 64*32256 = 2096640 floats
    assert call(_params(heads=1, seq=32289, dtype=0)) == -9
    assert call(_params(alpha=0.5)) == -2                         # the shared parameter checks still come first
    assert b"scratch" in lib.entmax_attn_strerror(-9)


def test_decode_entry_point_rejections(lib):
    from paper_2506_16640_b200.binding import DecodeParams

    def dparams(**kw):
        base = dict(batch=2, heads=4, q_len=2, kv_capacity=1000, head_dim=128, alpha=1.5, sm_scale=0.0, kv_stride_b=0,
                    kv_stride_h=0, kv_stride_n=0)
        base.update(kw)
        return DecodeParams(**base)

    p = dparams()
    need = lib.entmax_attn_decode_workspace_bytes(ctypes.byref(p))
    assert need >= 2 * 4 * 2 * 1000 * 4
    for bad in [dparams(q_len=0), dparams(q_len=9), dparams(kv_capacity=1), dparams(head_dim=96), dparams(alpha=1.0),
                dparams(alpha=100.0), dparams(kv_stride_b=8, kv_stride_h=8, kv_stride_n=64)]:
        assert lib.entmax_attn_decode_workspace_bytes(ctypes.byref(bad)) == 0
    fake, odd, nul = ctypes.c_void_p(4096), ctypes.c_void_p(4100), ctypes.c_void_p(0)
    call = lambda q, ws, nbytes, beta=None: lib.entmax_attn_decode_fwd(
        ctypes.byref(p), q, fake, fake, None, beta, None, None, None, fake, fake, None, ws, nbytes, None, None)
    assert call(nul, fake, 1 << 30) == -6
    assert call(odd, fake, 1 << 30) == -4
    assert call(fake, fake, 1 << 30, beta=fake) == -6          # beta without gamma/delta
    assert call(fake, fake, 16) == -5
    assert call(fake, nul, 1 << 30) == -5


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2506_16640_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(binding.EntmaxAttnError):
        binding.load()
