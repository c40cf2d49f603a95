"""CPU-only checks of the boundary: the shared library builds, loads and exports every
symbol the header declares; host-side argument validation answers without touching a GPU."""
import ctypes
import os
import re

import pytest

import paper_2601_16238_b200 as vt
from paper_2601_16238_b200 import build as vt_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "vt_attn.h")
SUITE_HEADER = os.path.join(ROOT, "include", "vt_suite.h")


@pytest.fixture(scope="module")
def lib():
    vt_build.build()
    return vt.load_library()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vt_attn_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_north_star_calls():
    names = declared_functions()
    for must in ("vt_attn_fwd", "vt_attn_bwd", "vt_attn_bwd_workspace_bytes", "vt_attn_abi_version"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), f"{name} is declared in vt_attn.h but not exported"


def test_binding_covers_every_declared_symbol():
    assert sorted(vt.EXPORTS) == declared_functions()


def declared_suite_functions():
    text = re.sub(r"/\*.*?\*/", "", open(SUITE_HEADER).read(), flags=re.S)
    return sorted(set(re.findall(r"\b(vt_suite_[a-z0-9_]+)\s*\(", text)))


def test_suite_header_symbols_are_exported_and_bound(lib):
    from paper_2601_16238_b200 import suite
    names = declared_suite_functions()
    assert "vt_suite_rmsnorm_fwd" in names and "vt_suite_layernorm_bwd" in names and "vt_suite_rope_apply" in names
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in vt_suite.h but not exported"
        assert callable(getattr(suite, name)), f"{name} has no binding"
    assert sorted(suite.SUITE_EXPORTS) == names


def test_suite_argument_validation_returns_before_any_cuda_call(lib):
    from paper_2601_16238_b200 import suite
    suite._lib()
    p = _fake()
    assert lib.vt_suite_rmsnorm_fwd(p, p, p, None, 4, 100, 1e-5, None) == vt.ERR_UNSUPPORTED           # cols % 8
    assert lib.vt_suite_rmsnorm_fwd(p, p, p, None, 4, 65544, 1e-5, None) == vt.ERR_UNSUPPORTED
    assert lib.vt_suite_rmsnorm_fwd(p, p, p, None, 0, 128, 1e-5, None) == vt.ERR_INVALID_ARGUMENT
    assert lib.vt_suite_rmsnorm_fwd(p, None, p, None, 4, 128, 1e-5, None) == vt.ERR_INVALID_ARGUMENT
    assert lib.vt_suite_rmsnorm_fwd(p, p, p, None, 4, 128, -1.0, None) == vt.ERR_INVALID_ARGUMENT
    assert lib.vt_suite_layernorm_fwd(p, p, p, _fake(0x1004), None, None, 4, 128, 1e-5, None) == vt.ERR_INVALID_ARGUMENT
    assert lib.vt_suite_layernorm_bwd_workspace_bytes(8192) == 2 * 148 * 8192 * 4
    assert lib.vt_suite_layernorm_bwd_workspace_bytes(1024) == 2 * 592 * 1024 * 4
    assert lib.vt_suite_layernorm_bwd_workspace_bytes(8200) == 0
    assert lib.vt_suite_layernorm_bwd(p, p, p, p, p, p, p, p, 4, 8192, p, 1024, None) == vt.ERR_WORKSPACE_TOO_SMALL
    assert lib.vt_suite_layernorm_bwd(p, p, p, p, p, p, p, p, 4, 16384, p, 1 << 30, None) == vt.ERR_UNSUPPORTED
    assert lib.vt_suite_rope_tables(p, p, 16, 24, 10000.0, None) == vt.ERR_UNSUPPORTED                  # D % 16
    assert lib.vt_suite_rope_tables(p, p, 16, 64, -1.0, None) == vt.ERR_INVALID_ARGUMENT
    assert lib.vt_suite_rope_apply(p, p, p, p, 0, 16, 64, 0, None) == vt.ERR_INVALID_ARGUMENT
    assert lib.vt_suite_rope_apply(p, p, p, p, 2, 16, 1024, 0, None) == vt.ERR_UNSUPPORTED


def test_abi_version_and_strings(lib):
    assert lib.vt_attn_abi_version() == 1
    assert lib.vt_attn_status_string(0) == b"ok"
    for code in (-1, -2, -3, -4, -5, -99):
        assert lib.vt_attn_status_string(code)


def test_info(lib):
    info = vt.vt_attn_get_info()
    assert info[0] == 1 and info[1] == 128 and info[2] == 64


def test_workspace_and_staging_sizes(lib):
    assert vt.vt_attn_bwd_workspace_bytes(1, 2, 2, 128, 128, 64) == 1024
    assert vt.vt_attn_bwd_workspace_bytes(128, 6, 6, 65, 65, 64) == (128 * 6 * 65 * 4 + 255) // 256 * 256
    assert vt.vt_attn_bwd_workspace_bytes(1, 3, 2, 128, 128, 64) == 0       # Hq % Hkv != 0
    assert vt.vt_attn_bwd_workspace_bytes(1, 2, 2, 128, 128, 100) == 0      # unsupported D (not a multiple of 8)
    assert vt.vt_attn_bwd_workspace_bytes(1, 2, 2, 128, 128, 96) == 1024     # any multiple of 8 up to 128
    assert vt.vt_attn_bwd_workspace_bytes(1, 2, 2, 128, 128, 136) == 1024    # and up to 256
    assert vt.vt_attn_bwd_workspace_bytes(1, 2, 2, 128, 128, 264) == 0
    assert vt.vt_attn_fwd_kernel_kind(1, 2, 2, 128, 128, 256, False) == 0       # forward only: up to 256
    assert vt.vt_attn_fwd_splitkv_plan(1, 8, 2, 1, 4096, 256)[0] >= 1
    # packed batches: equal cache lengths get the one-wave choice of the batched call, ragged ones more chunks
    even = vt.vt_attn_fwd_splitkv_plan(16, 32, 8, 1, 32768, 128)
    assert vt.vt_attn_fwd_splitkv_varlen_plan(16, 32, 8, 16 * 32768, 1, 32768, 128) == even
    ragged = vt.vt_attn_fwd_splitkv_varlen_plan(16, 32, 8, 16 * 20000, 1, 32768, 128)
    assert ragged[0] > even[0] and ragged[0] <= 16 and ragged[1] == even[1]
    assert vt.vt_attn_fwd_splitkv_varlen_plan(128, 32, 8, 128 * 4000, 1, 8192, 128)[0] == 4
    assert vt.vt_attn_fwd_splitkv_varlen_plan(16, 32, 8, 16 * 20000, 1, 32768, 128, 3)[0] == 3
    fwd = vt.vt_attn_host_staging_bytes(1, 2, 2, 128, 128, 64, False)
    both = vt.vt_attn_host_staging_bytes(1, 2, 2, 128, 128, 64, True)
    assert fwd == 4 * 32768 + 1024 and both > 2 * fwd - 2048


def _fake(addr=0x1000):
    return ctypes.c_void_p(addr)


def test_argument_validation_returns_before_any_cuda_call(lib):
    f = lib.vt_attn_fwd
    good = dict(B=1, Hq=2, Hkv=2, Sq=128, Sk=128, D=64)

    def call(q=_fake(), k=_fake(), v=_fake(), o=_fake(), lse=_fake(), causal=0, scale=0.125, **kw):
        d = dict(good, **kw)
        return f(q, k, v, o, lse, d["B"], d["Hq"], d["Hkv"], d["Sq"], d["Sk"], d["D"], causal, scale, None)

    assert call(B=0) == vt.ERR_INVALID_ARGUMENT
    assert call(Sk=0) == vt.ERR_INVALID_ARGUMENT
    assert call(Hq=3, Hkv=2) == vt.ERR_INVALID_ARGUMENT
    assert call(D=100) == vt.ERR_UNSUPPORTED
    assert call(D=264) == vt.ERR_UNSUPPORTED                         # the forward goes up to 256
    assert call(D=4) == vt.ERR_UNSUPPORTED
    assert call(scale=0.0) == vt.ERR_INVALID_ARGUMENT
    assert call(scale=float("nan")) == vt.ERR_INVALID_ARGUMENT
    assert call(scale=float("inf")) == vt.ERR_INVALID_ARGUMENT
    assert call(q=None) == vt.ERR_INVALID_ARGUMENT
    assert call(k=_fake(0x1008)) == vt.ERR_INVALID_ARGUMENT          # not 16-byte aligned
    assert call(Sq=(1 << 24) + 1) == vt.ERR_INVALID_ARGUMENT

    g = lib.vt_attn_bwd
    args = [_fake()] * 9 + [1, 2, 2, 128, 128, 64, 0, 0.125]
    assert g(*args, _fake(), 1023, None) == vt.ERR_WORKSPACE_TOO_SMALL
    assert g(*args, None, 4096, None) == vt.ERR_INVALID_ARGUMENT
    bad = [_fake()] * 9 + [1, 2, 2, 128, 128, 84, 0, 0.125]
    assert g(*bad, _fake(), 4096, None) == vt.ERR_UNSUPPORTED
    bad = [_fake()] * 9 + [1, 2, 2, 128, 128, 264, 0, 0.125]         # the backward goes up to 256 too
    assert g(*bad, _fake(), 4096, None) == vt.ERR_UNSUPPORTED
    wide = [_fake()] * 9 + [1, 2, 2, 128, 128, 192, 0, 0.125]
    assert g(*wide, _fake(), 16, None) == vt.ERR_WORKSPACE_TOO_SMALL  # 128 < D <= 256 is accepted: the next check answers
    assert vt.vt_attn_bwd_kernel_kind(1, 2, 2, 128, 128, 192) == 2 and vt.vt_attn_bwd_kernel_kind(1, 2, 2, 128, 128, 128) == 0
    assert vt.vt_attn_bwd_workspace_bytes(1, 2, 2, 128, 128, 256) == 1024
    assert lib.vt_attn_fwd_host(*([_fake()] * 5), 1, 2, 2, 128, 128, 64, 0, 0.125, _fake(0x10000), 16, None) \
        == vt.ERR_WORKSPACE_TOO_SMALL
    assert lib.vt_attn_selftest_timeout(0, None) == vt.ERR_INVALID_ARGUMENT
    # head dimensions above 128 exist only in the [B, H, S, D] forward and backward entry points and the host-buffer ones
    # built on them: the packed ones answer "unsupported", as does a V width outside [8, 256]
    cu = _fake(0x2000)
    assert lib.vt_attn_fwd_varlen(*([_fake()] * 5), cu, cu, 2, 2, 2, 256, 256, 128, 128, 192, 0, 0.1, None) == vt.ERR_UNSUPPORTED
    assert lib.vt_attn_fwd_host(*([_fake()] * 5), 1, 2, 2, 128, 128, 192, 0, 0.125, _fake(0x10000), 16, None) == vt.ERR_WORKSPACE_TOO_SMALL
    assert lib.vt_attn_fwd_host(*([_fake()] * 5), 1, 2, 2, 128, 128, 264, 0, 0.125, _fake(0x10000), 1 << 30, None) == vt.ERR_UNSUPPORTED
    assert vt.vt_attn_host_staging_bytes(1, 2, 2, 128, 128, 256, True) > vt.vt_attn_host_staging_bytes(1, 2, 2, 128, 128, 256, False) > 0
    assert vt.vt_attn_host_staging_bytes(1, 2, 2, 128, 128, 264, False) == 0
    assert lib.vt_attn_fwd_dv(*([_fake()] * 5), 1, 2, 2, 128, 128, 192, 264, 0, 0.125, None) == vt.ERR_UNSUPPORTED
    assert lib.vt_attn_fwd_dv(*([_fake()] * 5), 1, 2, 2, 128, 128, 192, 100, 0, 0.125, None) == vt.ERR_UNSUPPORTED


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    from paper_2601_16238_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    with pytest.raises(FileNotFoundError):
        binding.load_library(str(tmp_path / "nope.so"))


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2601_16238_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower() or f == "inputs.py", f"{f} mentions the oracle"


def test_status_word_kernel_ids_are_distinct():
    """A timed-out wait names its kernel in the low byte of the status word: two kernels must not share an id."""
    import re
    ids = {}
    csrc = os.path.join(ROOT, "paper_2601_16238_b200", "csrc")
    for f in sorted(os.listdir(csrc)):
        for name, val in re.findall(r"constexpr uint32_t (\w+_KERNEL_ID) = (\d+);", open(os.path.join(csrc, f)).read()):
            assert int(val) not in ids, f"{name} and {ids[int(val)]} share id {val}"
            assert 0 < int(val) < 256
            ids[int(val)] = name
    assert len(ids) >= 9


def test_splitkv_plan_and_workspace(lib):
    # decoding: 4 query heads per KV head, one query each -> the group shares a tile; 512 steps of 64 keys
    used, share = vt.vt_attn_fwd_splitkv_plan(4, 32, 8, 1, 32768, 128, 0)
    assert share and 1 <= used <= 128
    # one wave of two blocks per SM on 148 SMs: 32 (batch, KV head) pairs x used chunks
    assert 148 < 32 * used <= 296
    # an explicit request is honoured unless chunks would be empty
    assert vt.vt_attn_fwd_splitkv_plan(1, 2, 2, 128, 1024, 64, 4) == (4, False)
    assert vt.vt_attn_fwd_splitkv_plan(1, 2, 2, 128, 100, 64, 8) == (2, False)       # only two steps of 64 keys exist
    assert vt.vt_attn_fwd_splitkv_plan(1, 2, 2, 128, 64 * 5, 64, 4) == (3, False)    # chunks of 2 steps: 3 chunks cover 5 steps
    # long prefill already fills the GPU: no split by default
    assert vt.vt_attn_fwd_splitkv_plan(4, 16, 16, 8192, 8192, 128, 0)[0] == 1
    # heads share a tile only when (Hq / Hkv) * Sq <= 128 and there is a group at all
    assert vt.vt_attn_fwd_splitkv_plan(1, 8, 2, 32, 4096, 128, 0)[1] is True
    assert vt.vt_attn_fwd_splitkv_plan(1, 8, 2, 33, 4096, 128, 0)[1] is False
    assert vt.vt_attn_fwd_splitkv_plan(1, 8, 8, 1, 4096, 128, 0)[1] is False
    need = lib.vt_attn_fwd_splitkv_workspace_bytes(1, 2, 2, 128, 1024, 64, 4)
    rows = 1 * 2 * 128
    assert need == 4 * rows * 64 * 4 + (4 * rows * 4 + 255) // 256 * 256
    assert lib.vt_attn_fwd_splitkv_workspace_bytes(1, 2, 2, 128, 1024, 64, 129) == 0
    assert lib.vt_attn_fwd_splitkv_workspace_bytes(1, 3, 2, 128, 1024, 64, 2) == 0


def test_forward_kernel_choice(lib):
    # long D = 128 sequences with enough blocks: the two-tile kernel; everything else the one-tile kernel
    assert vt.vt_attn_fwd_kernel_kind(4, 16, 16, 8192, 8192, 128, False) == 1
    assert vt.vt_attn_fwd_kernel_kind(4, 16, 16, 2048, 2048, 128, False) == 1
    assert vt.vt_attn_fwd_kernel_kind(4, 16, 16, 2048, 2048, 128, True) == 0      # causal: from 32 tiles on
    assert vt.vt_attn_fwd_kernel_kind(4, 16, 16, 4096, 4096, 128, True) == 1
    assert vt.vt_attn_fwd_kernel_kind(4, 16, 16, 4096, 4096, 64, False) == 0      # D = 64
    assert vt.vt_attn_fwd_kernel_kind(1, 4, 4, 8192, 8192, 128, False) == 0        # 4 heads x 32 pairs = 128 blocks < 148 SMs
    assert vt.vt_attn_fwd_kernel_kind(1, 5, 5, 8192, 8192, 128, False) == 1        # 160 blocks
    # causal shapes whose blocks of two tiles fill the SMs in one even wave get the two-tiles-in-sequence kernel
    assert vt.vt_attn_fwd_kernel_kind(4, 16, 16, 1024, 1024, 128, True) == 2       # 64 heads x 4 pairs = 256 blocks
    assert vt.vt_attn_fwd_kernel_kind(1, 74, 74, 1024, 1024, 64, True) == 2        # 296 blocks
    assert vt.vt_attn_fwd_kernel_kind(1, 80, 80, 1024, 1024, 128, True) == 0       # 320 blocks: a second wave
    assert vt.vt_attn_fwd_kernel_kind(1, 40, 40, 1024, 1024, 128, True) == 0       # 160 blocks: uneven over 148 SMs
    assert vt.vt_attn_fwd_kernel_kind(1, 32, 32, 1024, 1024, 128, True) == 0       # 128 blocks: one per SM is no better than the one-tile kernel
    assert vt.vt_attn_fwd_kernel_kind(1, 60, 60, 1024, 1024, 128, True) == 2       # 240 blocks: the window starts here
    assert vt.vt_attn_fwd_kernel_kind(1, 59, 59, 1024, 1024, 128, True) == 0
    assert vt.vt_attn_fwd_kernel_kind(1, 36, 36, 2048, 2048, 128, True) == 0       # sixteen tiles per head
    assert vt.vt_attn_fwd_kernel_kind(1, 48, 48, 1536, 1536, 128, True) == 2       # twelve
    assert vt.vt_attn_fwd_kernel_kind(8, 8, 8, 256, 256, 64, True) == 0            # 128 one-tile blocks already fit
    assert vt.vt_attn_fwd_kernel_kind(4, 16, 16, 1024, 1024, 128, False) == 0      # not causal
    assert vt.vt_attn_fwd_kernel_kind(4, 16, 16, 1024, 2048, 128, 2) == 0          # bottom-right with Sk != Sq
    assert vt.vt_attn_fwd_kernel_kind(4, 16, 16, 1024, 1024, 128, 2) == 2          # ... with Sk == Sq: the same mask


# ------------------------------------------------------------------------------------------------
# The binding checks every tensor's shape against the others before the library is entered (the kernels trust the sizes
# they are told).  Shapes are checked before devices, so CPU tensors reach these checks without a GPU.
# ------------------------------------------------------------------------------------------------
def _t(*shape, dtype=None):
    import torch
    return torch.zeros(*shape, dtype=dtype or torch.bfloat16)


@pytest.mark.parametrize("bad", ["v_short", "v_heads", "k_batch", "k_dim", "gqa", "o_shape", "lse_shape", "rank"])
def test_forward_binding_rejects_mismatched_shapes(lib, bad):
    import torch
    q, k, v = _t(2, 4, 10, 64), _t(2, 2, 12, 64), _t(2, 2, 12, 64)
    o = lse = None
    if bad == "v_short":
        v = _t(2, 2, 11, 64)
    elif bad == "v_heads":
        v = _t(2, 1, 12, 64)
    elif bad == "k_batch":
        k = _t(1, 2, 12, 64)
    elif bad == "k_dim":
        k = _t(2, 2, 12, 32)
    elif bad == "gqa":
        k, v = _t(2, 3, 12, 64), _t(2, 3, 12, 64)
    elif bad == "o_shape":
        o = _t(2, 4, 9, 64)
    elif bad == "lse_shape":
        lse = _t(2, 4, 9, dtype=torch.float32)
    elif bad == "rank":
        q = _t(2, 40, 64)
    with pytest.raises(ValueError, match="shape|disagree|multiple|match|must be"):
        vt.vt_attn_fwd(q, k, v, False, 0.125, o, lse)
    if bad not in ("rank",):
        with pytest.raises(ValueError, match="shape|disagree|multiple|match|must be"):
            vt.vt_attn_fwd_splitkv(q, k, v, False, 0.125, 2, o, lse)


@pytest.mark.parametrize("bad", ["o", "d_o", "lse", "dq", "dk", "dv", "v"])
def test_backward_binding_rejects_mismatched_shapes(lib, bad):
    import torch
    q, k, v = _t(1, 4, 10, 64), _t(1, 2, 12, 64), _t(1, 2, 12, 64)
    args = dict(o=_t(1, 4, 10, 64), d_o=_t(1, 4, 10, 64), lse=_t(1, 4, 10, dtype=torch.float32), dq=None, dk=None, dv=None)
    wrong = {"o": _t(1, 4, 9, 64), "d_o": _t(1, 4, 10, 32), "lse": _t(1, 4, 11, dtype=torch.float32), "dq": _t(1, 4, 9, 64),
             "dk": _t(1, 2, 11, 64), "dv": _t(1, 2, 12, 32)}
    if bad == "v":
        v = _t(1, 2, 13, 64)
    else:
        args[bad] = wrong[bad]
    with pytest.raises(ValueError, match="shape|match"):
        vt.vt_attn_bwd(q, k, v, args["o"], args["d_o"], args["lse"], True, 0.125, args["dq"], args["dk"], args["dv"])
    full = {n: (t if t is not None else _t(*{"dq": q, "dk": k, "dv": v}[n].shape)) for n, t in args.items()}
    if bad == "v":
        full["dv"] = _t(1, 2, 12, 64)
    with pytest.raises(ValueError, match="shape|match"):
        vt.vt_attn_bwd_static_scratch(q, k, v, full["o"], full["d_o"], full["lse"], True, 0.125, full["dq"], full["dk"], full["dv"])


def test_packed_and_host_bindings_reject_mismatched_shapes(lib):
    import torch
    q, k, v = _t(30, 4, 64), _t(40, 2, 64), _t(39, 2, 64)
    cu = torch.tensor([0, 10, 30], dtype=torch.int32)
    with pytest.raises(ValueError, match="shape"):
        vt.vt_attn_fwd_varlen(q, k, v, cu, cu, 20, 20, True, 0.125)
    v = _t(40, 2, 64)
    with pytest.raises(ValueError, match="shape"):
        vt.vt_attn_fwd_varlen(q, k, v, cu, cu, 20, 20, True, 0.125, lse=_t(30, 4, dtype=torch.float32))
    with pytest.raises(ValueError, match="shape"):
        vt.vt_attn_bwd_varlen(q, k, v, _t(30, 4, 64), _t(29, 4, 64), _t(4, 30, dtype=torch.float32), cu, cu, 20, 20, True, 0.125)
    # host-buffer entry points: host tensors are what they take, so every check is reachable here
    hq, hk, hv = _t(1, 2, 8, 64), _t(1, 2, 8, 64), _t(1, 2, 7, 64)
    stage = torch.zeros(1024, dtype=torch.uint8)
    with pytest.raises(ValueError, match="match"):
        vt.vt_attn_fwd_host(hq, hk, hv, _t(1, 2, 8, 64), _t(1, 2, 8, dtype=torch.float32), False, 0.125, stage)
    with pytest.raises(ValueError, match="shape"):
        vt.vt_attn_fwd_host(hq, hk, hk, _t(1, 2, 9, 64), _t(1, 2, 8, dtype=torch.float32), False, 0.125, stage)
    with pytest.raises(ValueError, match="shape"):
        vt.vt_attn_merge_partial(_t(4, 64, dtype=torch.float32), _t(5, dtype=torch.float32), _t(4, 64), _t(4, dtype=torch.float32), True)
