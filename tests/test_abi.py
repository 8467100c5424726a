"""The C-ABI library loads and exports every symbol the header declares; host-side validation
rejects bad arguments before anything is launched (no GPU needed)."""
import ctypes
import re
from pathlib import Path

import pytest

from paper_2603_06738_b200 import binding, build

ROOT = Path(__file__).resolve().parent.parent
HEADER = (ROOT / "include" / "rib_window_attn.h").read_text()


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.library()


def declared_functions():
    text = re.sub(r"/\*.*?\*/", "", HEADER, flags=re.S)
    return sorted(set(re.findall(r"\b(rib_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_functions()
    assert set(binding.EXPORTS) <= set(names)
    assert len(names) >= 7
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in the header but not exported"


def test_status_strings(lib):
    for code in range(-7, 1):
        s = binding.rib_status_string(code)
        assert s and "unknown" not in s
    assert "unknown" in binding.rib_status_string(-99)


def fwd_args(**over):
    a = dict(q=256, k=512, v=768, pq=1024, pk=1280, B=1, H=32, W=32, heads=2, d=32, r=16, window=16,
             shift=0, out=2048, lse=4096, stream=None)
    a.update(over)
    return [a[k] for k in ("q", "k", "v", "pq", "pk", "B", "H", "W", "heads", "d", "r", "window", "shift",
                           "out", "lse", "stream")]


@pytest.mark.parametrize("over,code", [
    (dict(q=None), -1), (dict(out=None), -1), (dict(pq=None), -1),
    (dict(H=40), -2), (dict(shift=16), -2), (dict(shift=-1), -2), (dict(B=0), -2), (dict(window=0), -2),
    (dict(d=128), -3), (dict(r=72), -3), (dict(d=65), -3),
    (dict(k=516), -4), (dict(lse=4100), -4),
])
def test_fwd_rejects_bad_arguments_without_launching(lib, over, code):
    """Validation order: NULL, shape, support, alignment; fake pointers are never dereferenced."""
    assert lib.rib_window_attn_fwd(*fwd_args(**over)) == code


def headwise_args(stride, **over):
    a = fwd_args(**over)
    return a[:5] + [stride] + a[5:]


def test_headwise_and_padded_entry_points_validate_before_any_cuda_call(lib):
    n_r = 16 * 16 * 16
    # stride: 0 (shared table) or a multiple of 8 that is at least n * r
    for stride, code in ((n_r - 8, -2), (n_r + 4, -2), (-8, -2)):
        assert lib.rib_window_attn_fwd_headwise(*headwise_args(stride)) == code
        assert lib.rib_window_attn_fwd_padded(*headwise_args(stride)) == code
        assert lib.rib_window_attn_bwd_headwise_workspace(stride, 1, 32, 32, 2, 32, 16, 16) == 0
    # only the padded entry point takes maps that are not multiples of the window; the other checks stay
    assert lib.rib_window_attn_fwd_headwise(*headwise_args(0, H=40)) == -2
    assert lib.rib_window_attn_fwd_padded(*headwise_args(0, H=40, q=None)) == -1
    assert lib.rib_window_attn_fwd_padded(*headwise_args(0, H=40, shift=16)) == -2
    assert lib.rib_window_attn_fwd_padded(*headwise_args(0, H=0)) == -2
    assert lib.rib_window_attn_fwd_padded(*headwise_args(0, H=40, d=72)) == -3
    assert lib.rib_window_attn_fwd_padded(*headwise_args(0, H=40, v=770)) == -4
    # backward on maps that are not multiples of the window: sized by the windows of the extended map on the tcgen05
    # shapes, one float per token-head on the any-shape kernels
    assert lib.rib_window_attn_bwd_padded_workspace(0, 1, 40, 56, 2, 32, 16, 16) >= 264 * 48 * 64 * 2
    assert lib.rib_window_attn_bwd_padded_workspace(0, 1, 41, 56, 2, 32, 16, 16) == (4 * 41 * 56 * 2 + 255) // 256 * 256
    assert lib.rib_window_attn_bwd_padded_workspace(0, 1, 32, 32, 2, 32, 16, 16) == lib.rib_window_attn_bwd_workspace(1, 32, 32, 2, 32, 16, 16)
    assert lib.rib_window_attn_bwd_padded_workspace(0, 1, 0, 56, 2, 32, 16, 16) == 0
    # rank 32 needs a larger backward workspace than rank 16 on the tcgen05 shapes
    assert lib.rib_window_attn_bwd_workspace(1, 32, 32, 2, 32, 32, 16) > lib.rib_window_attn_bwd_workspace(1, 32, 32, 2, 32, 16, 16)
    assert (lib.rib_window_attn_bwd_headwise_workspace(2 * n_r, 1, 32, 32, 2, 32, 16, 16)
            > lib.rib_window_attn_bwd_headwise_workspace(0, 1, 32, 32, 2, 32, 16, 16))


def test_bwd_rejects_bad_arguments(lib):
    base = dict(q=256, k=512, v=768, pq=1024, pk=1280, out=1536, lse=1792, dout=2048, B=1, H=32, W=32, heads=2,
                d=32, r=16, window=16, shift=0, dq=4096, dk=8192, dv=12288, dpq=16384, dpk=20480,
                ws=65536, ws_bytes=1 << 20, stream=None)
    order = ("q", "k", "v", "pq", "pk", "out", "lse", "dout", "B", "H", "W", "heads", "d", "r", "window", "shift",
             "dq", "dk", "dv", "dpq", "dpk", "ws", "ws_bytes", "stream")

    def call(**over):
        a = dict(base); a.update(over)
        return lib.rib_window_attn_bwd(*[a[k] for k in order])

    assert call(lse=None) == -1
    assert call(dpq=None) == -1
    assert call(W=33) == -2
    assert call(r=72) == -3
    assert call(dv=12290) == -4
    assert call(ws=None) == -5
    assert call(ws_bytes=16) == -5
    assert call(ws=65536 + 16) == -4
    need = lib.rib_window_attn_bwd_workspace(1, 32, 32, 2, 32, 16, 16)
    assert need >= 4 * 32 * 32 * 2 and need % 256 == 0
    assert lib.rib_window_attn_bwd_workspace(1, 33, 32, 2, 32, 16, 16) == 0


def test_path_knob(lib):
    assert binding.rib_set_path(binding.RIB_PATH_GENERIC) in (0, 1)
    assert binding.rib_set_path(binding.RIB_PATH_NONE) == binding.RIB_PATH_GENERIC
    assert binding.rib_set_path(77) == binding.RIB_PATH_NONE   # invalid value: unchanged


def test_cla_backward_entry_points_validate_before_any_cuda_call(lib):
    a = [256, 512, 768, 1024, 1280, 1536]                       # x, w_dw, b_dw, w_pw, b_pw, dgate
    outs = [2048, 4096, 8192, 12288, 16384]                     # dx, dw_dw, db_dw, dw_pw, db_pw
    need = lib.rib_cla_gate_bwd_workspace(1, 5, 7, 64)
    assert need == (5 * 7 * 64 + 64 * 64) * 4
    assert lib.rib_cla_gate_bwd_workspace(1, 0, 7, 64) == 0
    call = lambda **kw: lib.rib_cla_gate_bwd(*kw.get("ins", a), kw.get("B", 1), 5, 7, kw.get("D", 64), *kw.get("outs", outs),
                                             kw.get("ws", 32768), kw.get("ws_bytes", need), None)
    assert call(ins=[None] + a[1:]) == -1
    assert call(outs=outs[:4] + [None]) == -1
    assert call(B=0) == -2
    assert call(D=95) == -3                                                        # an odd channel count
    assert call(D=200) == -3                                                       # more than 192 channels
    assert lib.rib_cla_gate_bwd_workspace(1, 5, 7, 96) == (5 * 7 * 128 + 128 * 128) * 4   # 96 channels run as 128
    assert call(outs=[2050] + outs[1:]) == -4
    assert call(ws=None) == -5
    assert call(ws_bytes=need - 1) == -5
    assert lib.rib_cla_product(256, 512, 12, 768, None) == -2                      # count not a multiple of 8
    assert lib.rib_cla_product(256, None, 16, 768, None) == -1
    assert lib.rib_cla_product(256, 520, 16, 768, None) == -4
    assert lib.rib_cla_product(256, 512, 0, 768, None) == 0                        # nothing to do
    assert lib.rib_cla_product_bwd(256, 512, 768, -8, 1024, 1280, None) == -2
    assert lib.rib_cla_product_bwd(256, 512, None, 16, 1024, 1280, None) == -1
    assert lib.rib_cla_product_bwd(256, 512, 768, 16, 1024, 1284, None) == -4
