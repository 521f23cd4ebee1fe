"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "flat_attn.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2107_06419_b200 import build
    return ctypes.CDLL(build.build())


@pytest.fixture(scope="module")
def api(lib):
    from paper_2107_06419_b200 import api as _api
    return _api


def declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(flat_(?:attn|qkv_proj|out_proj|fc|layernorm)_\w+)\s*\(", src)))


def test_header_declares_and_library_exports(lib, api):
    names = declared_functions()
    assert "flat_attn_fwd" in names and "flat_attn_naive_fwd" in names and len(names) >= 9
    for n in names:
        assert hasattr(lib, n), "library does not export " + n
    assert sorted(api.EXPORTS) == [n for n in names if n != "flat_attn_params"]
    for n in api.EXPORTS:
        assert callable(getattr(api, n)), "binding lacks " + n


def test_status_strings_and_version(api):
    assert api.flat_attn_version() >= 100
    seen = {api.flat_attn_status_string(c) for c in range(8)}
    assert len(seen) == 8 and api.flat_attn_status_string(0) == "ok"
    assert api.flat_attn_status_string(99) == "unknown status"


def _params(api, **kw):
    p = api.flat_attn_params_t()
    p.Q, p.K, p.V, p.O = 0x10000, 0x20000, 0x30000, 0x40000     # never dereferenced on the host
    p.B, p.H, p.Nq, p.Nk, p.d = 1, 2, 128, 128, 64
    p.scale, p.dtype, p.variant = 0.125, 0, 0
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def test_projection_argument_errors(api):
    # (no GPU needed: every case is rejected before a launch)
    f = api._lib.flat_qkv_proj_fwd
    ok = dict(X=0x10000, W=0x20000, Q=0x30000, K=0x40000, V=0x50000, B=2, N=256, H=4, d=64, Dm=256)
    def qkv(**kw):
        a = dict(ok, **kw)
        return f(a["X"], a["W"], a["Q"], a["K"], a["V"], a["B"], a["N"], a["H"], a["d"], a["Dm"], None, None)
    assert qkv(X=None) == 1 and qkv(V=None) == 1
    assert qkv(B=0) == 2 and qkv(N=-1) == 2 and qkv(B=2 ** 20, N=2 ** 20) == 2
    assert qkv(d=32) == 3 and qkv(H=3) == 3 and qkv(Dm=200) == 3        # H*d must be a multiple of 256, Dm of 64
    assert qkv(X=0x10008) == 4
    g = api._lib.flat_out_proj_fwd
    def outp(**kw):
        a = dict(dict(O=0x10000, W=0x20000, Y=0x30000, B=2, N=256, H=4, d=64, Dm=256), **kw)
        return g(a["O"], a["W"], a["Y"], a["B"], a["N"], a["H"], a["d"], a["Dm"], None, None)
    assert outp(Y=None) == 1 and outp(H=0) == 2
    assert outp(N=200) == 3 and outp(Dm=320) == 3 and outp(d=16) == 3   # N multiple of 128, Dm of 256
    assert outp(W=0x20004) == 4
    fc = api._lib.flat_fc_fwd
    assert fc(None, 0x20000, 0x30000, 128, 64, 256, None, None) == 1
    assert fc(0x10000, 0x20000, 0x30000, 0, 64, 256, None, None) == 2
    assert fc(0x10000, 0x20000, 0x30000, 128, 100, 256, None, None) == 3 and fc(0x10000, 0x20000, 0x30000, 128, 64, 128, None, None) == 3
    assert fc(0x10000, 0x20000, 0x30008, 128, 64, 256, None, None) == 4
    ln = api._lib.flat_layernorm_fwd
    assert ln(None, None, 0x20000, 0x30000, 0x40000, 16, 256, 1e-5, None) == 1
    assert ln(0x10000, None, 0x20000, 0x30000, 0x40000, 0, 256, 1e-5, None) == 2
    assert ln(0x10000, None, 0x20000, 0x30000, 0x40000, 16, 256, -1.0, None) == 2
    assert ln(0x10000, None, 0x20000, 0x30000, 0x40000, 16, 100, 1e-5, None) == 3      # D a multiple of 8
    assert ln(0x10000, None, 0x20000, 0x30000, 0x40000, 16, 16384, 1e-5, None) == 3    # D at most 8192
    assert ln(0x10000, 0x50008, 0x20000, 0x30000, 0x40000, 16, 256, 1e-5, None) == 4
    h = api._lib.flat_attn_layer_fwd
    def layer(**kw):
        a = dict(dict(X=0x10000, Wqkv=0x20000, Wo=0x30000, Y=0x40000, Q=0x50000, K=0x60000, V=0x70000, O=0x80000,
                      B=2, N=256, H=4, d=64, Dm=256, scale=0.125, causal=0), **kw)
        return h(a["X"], a["Wqkv"], a["Wo"], a["Y"], a["Q"], a["K"], a["V"], a["O"], a["B"], a["N"], a["H"], a["d"],
                 a["Dm"], a["scale"], a["causal"], None, None)
    assert layer(O=None) == 1 and layer(Wo=None) == 1
    assert layer(scale=float("nan")) == 2 and layer(B=0) == 2
    assert layer(N=200) == 3 and layer(causal=2) == 3 and layer(H=2) == 3
    assert layer(Y=0x40002) == 4


@pytest.mark.parametrize("kw,code", [
    (dict(Q=None), 1), (dict(O=None), 1),
    (dict(B=0), 2), (dict(Nk=-3), 2), (dict(scale=float("inf")), 2), (dict(scale=float("nan")), 2),
    (dict(B=70000), 2), (dict(B=60000, Nq=2 ** 31 - 1, Nk=2 ** 31 - 1), 2),
    (dict(d=48), 3), (dict(d=256), 3), (dict(dtype=2), 3), (dict(variant=9, dtype=1), 3),
    (dict(dtype=1, variant=2), 3), (dict(dtype=1, variant=3), 3), (dict(d=16, variant=3), 3), (dict(d=128, variant=4), 3), (dict(variant=7), 3), (dict(variant=17), 3), (dict(variant=15, d=32), 3), (dict(variant=16, d=128), 3), (dict(variant=11, d=128), 3), (dict(variant=14, dtype=1), 3), (dict(variant=8, d=32), 3), (dict(variant=10, dtype=1), 3), (dict(dtype=1, variant=7, d=128), 3), (dict(dtype=1, variant=7, d=32), 3), (dict(variant=6, Nk=513), 3), (dict(variant=6, d=128), 3), (dict(variant=6, dtype=1), 3), (dict(dtype=1, variant=5), 3), (dict(d=32, variant=5), 3), (dict(d=128, variant=5), 3), (dict(causal=2), 3), (dict(causal=-1), 3), (dict(causal=1, variant=2), 3), (dict(causal=1, variant=2, d=128), 3),                               # tensor-core kernel is bf16 only
    (dict(d=32, variant=2), 3),
    (dict(K=0x20008), 4), (dict(k_valid_len=0x50002), 4),
])
def test_fused_argument_errors(lib, api, kw, code):
    p = _params(api, **kw)
    assert api._lib.flat_attn_fwd_ex(ctypes.byref(p), None) == code
    assert api._lib.flat_attn_fwd_ex(None, None) == 1


def test_naive_and_host_argument_errors(api):
    p = _params(api)
    assert api._lib.flat_attn_naive_fwd_ex(ctypes.byref(p), None, 0x60000, None) == 1
    assert api._lib.flat_attn_naive_fwd_ex(ctypes.byref(p), 0x60004, 0x70000, None) == 4
    assert api._lib.flat_attn_naive_fwd(0x10000, 0x20000, 0x30000, 0x40000, 0x50000, 0x60000, 1, 1, 0, 5, 64, 1.0, None) == 2
    # the baseline's row softmax uses one thread block per row: more than 2^31 - 1 rows are refused up front
    rows = _params(api, B=4, H=1, Nq=2 ** 29, Nk=8)
    assert api._lib.flat_attn_naive_fwd_ex(ctypes.byref(rows), 0x60000, 0x70000, None) == 2
    assert api._lib.flat_attn_naive_fwd_ex(ctypes.byref(_params(api, B=2, H=1, Nq=2 ** 30, Nk=8)), 0x60000, 0x70000, None) == 2
    need = api.flat_attn_host_workspace_bytes(1, 2, 128, 128, 64)
    assert need == 4 * 2 * 128 * 64 * 2 + 256
    assert api.flat_attn_host_workspace_bytes(1, 2, 128, 128, 64, 1) == 4 * 2 * 128 * 64 * 4 + 256
    assert api.flat_attn_host_workspace_bytes(0, 2, 128, 128, 64) == 0
    assert api._lib.flat_attn_fwd_host(ctypes.byref(p), None, need, None) == 1
    assert api._lib.flat_attn_fwd_host(ctypes.byref(p), 0x100010, need, None) == 4
    assert api._lib.flat_attn_fwd_host(ctypes.byref(p), 0x100000, need - 1, None) == 5


def test_device_error_word_and_last_variant_calls(api):
    # host-side behaviour only: a NULL output pointer is refused, and before any fused call the last variant is 0
    assert api._lib.flat_attn_last_device_error(None) == 1
    import subprocess
    import sys
    r = subprocess.run([sys.executable, "-c",
                        "import paper_2107_06419_b200.api as a; print(a.flat_attn_last_variant())"],
                       cwd=ROOT, capture_output=True, text=True)
    assert r.returncode == 0 and r.stdout.strip() == "0", r.stderr


def test_binding_rejects_bad_tensors(api):
    import torch
    q = torch.zeros(1, 1, 4, 64, dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        api.flat_attn_fwd(q, q, q, q, 1.0)                      # host tensors on the device entry point
    with pytest.raises(TypeError):
        api._params(q.to(torch.float16), q, q, q, 1.0, None, None, 0, host=True)
    with pytest.raises(ValueError):
        api._params(q, q[:, :, :, :32], q, q, 1.0, None, None, 0, host=True)


def test_missing_library_fails_loudly(tmp_path):
    """Importing the binding without the built library raises; nothing falls back to the CPU."""
    import subprocess
    import sys
    pkg = tmp_path / "paper_2107_06419_b200"
    pkg.mkdir()
    for f in ("__init__.py", "api.py"):
        (pkg / f).write_text(open(os.path.join(ROOT, "paper_2107_06419_b200", f)).read())
    r = subprocess.run([sys.executable, "-c", "import paper_2107_06419_b200.api"], cwd=tmp_path,
                       capture_output=True, text=True, env={**os.environ, "PYTHONPATH": str(tmp_path)})
    assert r.returncode != 0 and "libflat_attn.so is not built" in r.stderr


def test_product_path_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2107_06419_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower() or f == "inputs.py", f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".cpp")):
            assert "paper_2107_06419_b200" not in open(os.path.join(ROOT, "oracle", f)).read()
