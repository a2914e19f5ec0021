"""CPU-only checks: the library builds, loads, exports what include/dppo.h declares, and rejects misuse
before anything is launched."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2602_04879_b200 import build
    build.build_library()
    from paper_2602_04879_b200 import binding as b
    return b


def declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            src = open(os.path.join(ROOT, "include", fn)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(dppo_[a-z0-9_]+)\s*\(", src))
    return sorted(names)


def test_every_declared_symbol_is_exported(binding):
    names = declared_functions()
    assert "dppo_loss_fwd_bwd" in names and "dppo_workspace_bytes" in names and len(names) >= 6
    lib = binding.lib()
    for n in names:
        assert hasattr(lib, n), n
    assert binding.version() >= 100


def test_options_struct_and_workspace_sizes(binding):
    """The binding's copy of dppo_opts has the library's size and field order (the header's struct, field by field), and
    the fused variant's workspace in row-block mode depends on the block, not on T."""
    B = binding
    assert int(B.lib().dppo_opts_size()) == ctypes.sizeof(B.DppoOpts)
    hdr = open(os.path.join(ROOT, "include", "dppo.h")).read()
    body = re.sub(r"/\*.*?\*/", "", hdr[hdr.index("typedef struct dppo_opts {"):hdr.index("} dppo_opts;")], flags=re.S)
    fields = re.findall(r"\b(?:float|int)\s+([a-z_]+)\s*;", body)
    assert fields == [f[0] for f in B.DppoOpts._fields_]
    d, V = 2048, 151936
    whole, block = B.dppo_fused_workspace_bytes(8192, d, V), B.dppo_fused_workspace_bytes(2048, d, V)
    assert whole > 2.5e9 and block < 0.9e9 and B.dppo_fused_workspace_bytes(2048, d, V, 20) - block > 2 * d * V - 4096
    assert B.dppo_fused_workspace_bytes(-1, d, V) == 0


def test_error_strings(binding):
    seen = set()
    for code in range(0, -13, -1):
        s = binding.error_string(code)
        assert s and s != "unknown error code"
        seen.add(s)
    assert len(seen) == 13
    assert binding.error_string(-99) == "unknown error code"


def test_workspace_bytes(binding):
    assert binding.dppo_workspace_bytes(0) == 256
    assert binding.dppo_workspace_bytes(1) == 256 + 3 * 256
    assert binding.dppo_workspace_bytes(16384) == 256 + 3 * 65536
    assert binding.dppo_workspace_bytes(65) == 256 + 3 * 512
    assert binding.dppo_workspace_bytes(65, 151936, 64, binding.TOPK_KL) == 256 + 3 * 512       # a function of T alone today
    assert binding.dppo_host_staging_bytes(0, 10, 0, 0) == 0
    a = binding.dppo_host_staging_bytes(128, 4096, 0, binding.BF16)
    b = binding.dppo_host_staging_bytes(128, 4096, 0, binding.BF16, dlogits_f32=True)
    assert b - a == 2 * 128 * 4096 * 4 and a > 2 * 128 * 4096 * 2


def _call(binding, **over):
    """dppo_loss_fwd_bwd with fake (never dereferenced) pointers; only host validation runs."""
    p = ctypes.c_void_p
    a = dict(logits=0x10000, T=4, V=64, ld=64, dt=binding.BF16, ids=0x20000, mu=0x30000, tk_ids=None, tk_p=None,
             adv=0x40000, tok=None, variant=0, K=0, delta=0.2, opts=None, loss=0x50000, D=0x60000, M=0x70000,
             dl=0x80000, ld_out=64, stats=None, status=0x90000, ws=0xA0000, ws_bytes=1 << 20)
    a.update(over)
    opts = a["opts"]
    return binding.lib().dppo_loss_fwd_bwd(p(a["logits"]), a["T"], a["V"], a["ld"], a["dt"], p(a["ids"]), p(a["mu"]),
                                           p(a["tk_ids"]), p(a["tk_p"]), p(a["adv"]), p(a["tok"]), a["variant"], a["K"],
                                           a["delta"], ctypes.byref(opts) if opts is not None else None, p(a["loss"]),
                                           p(a["D"]), p(a["M"]), p(a["dl"]), a["ld_out"], p(a["stats"]), p(a["status"]),
                                           p(a["ws"]), a["ws_bytes"], None)


def test_misuse_is_rejected_before_launch(binding):
    B = binding
    assert _call(B, T=-1) == -2
    assert _call(B, V=0) == -2
    assert _call(B, variant=2, K=65, tk_ids=1 << 8, tk_p=1 << 9) == -2
    assert _call(B, K=-1) == -2
    assert _call(B, dt=7) == -3
    assert _call(B, opts=B.DppoOpts(0.0, 5, 0, 0.0, 0.0)) == -3
    assert _call(B, variant=7) == -4
    assert _call(B, variant=-1) == -4
    assert _call(B, opts=B.DppoOpts(0.0, 0, 9, 0.0, 0.0)) == -11
    assert _call(B, logits=None) == -1
    assert _call(B, loss=None) == -1
    assert _call(B, status=None) == -1
    assert _call(B, mu=None) == -1
    assert _call(B, variant=3, K=4) == -5
    assert _call(B, variant=3, K=4, tk_ids=1 << 8) == -5
    assert _call(B, ld=63) == -6
    assert _call(B, ld_out=10) == -6
    assert _call(B, logits=0x10001) == -7
    assert _call(B, ws=None) == -8
    assert _call(B, ws=0xA0010) == -8
    assert _call(B, ws_bytes=100) == -8
    assert _call(B, dl=0x10000, opts=B.DppoOpts(0.0, B.DLOGITS_F32, 0, 0.0, 0.0)) == -9
    assert _call(B, dl=0x10000, ld_out=128) == -9
    # dlogits may be the logits buffer itself (in place) or a disjoint one; any other overlap is refused, for every kernel
    row = 64 * 2
    for kern in (B.KERNEL_AUTO, B.KERNEL_GENERIC, B.KERNEL_RING):
        o = B.DppoOpts(0.0, 0, kern, 0.0, 0.0)
        assert _call(B, dl=0x10000 + row, opts=o) == -9         # shifted by one row
        assert _call(B, dl=0x10000 + 3 * row + 32, opts=o) == -9    # starts inside the last row
        assert _call(B, dl=0x10000 - 2 * row, opts=o) == -9     # ends inside the logits
        assert _call(B, logits=0x10000, ld=128, dl=0x10000 + row, ld_out=128, opts=o) == -9   # interleaved rows of one allocation
    assert _call(B, opts=B.DppoOpts(0.0, 0, 0, 0.0, 0.0, 0, 0, 0, -5)) == -11      # negative wait limit
    for bad in (-1, 3, 8):                                                          # SMs per row: 0 (automatic), 1, 2 or 4
        assert _call(B, opts=B.DppoOpts(row_cluster=bad)) == -11
    # forcing the bulk-copy kernel on a layout it cannot take
    assert _call(B, V=63, ld=63, ld_out=64, opts=B.DppoOpts(0.0, 0, B.KERNEL_RING, 0.0, 0.0)) == -7     # rows shifted differently
    assert _call(B, logits=0x10002, opts=B.DppoOpts(0.0, 0, B.KERNEL_RING, 0.0, 0.0)) == -7


def test_missing_library_fails_loudly(binding, monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()


def test_product_does_not_import_oracle():
    pkg = os.path.join(ROOT, "paper_2602_04879_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower(), f
