"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every declared
symbol, sizes workspaces sensibly and rejects bad arguments before anything is launched."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ex():
    from paper_2608_24938_b200 import build
    build.build()
    from paper_2608_24938_b200 import binding
    return binding


def declared_functions():
    src = open(os.path.join(ROOT, "include", "exfold.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(exfold_[a-z0-9_]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(ex):
    names = declared_functions()
    assert set(ex.EXPORTS) == set(names)
    for n in names:
        assert hasattr(ex.lib, n), n


def test_status_strings(ex):
    for code in (0, -1, -2, -3, -4, -5, 1):
        assert ex.exfold_status_string(code) not in ("", "unknown status")
    assert ex.exfold_status_string(12345) == "unknown status"


def test_workspace_sizes(ex):
    qwen = ex.make_layer(128, 0, 2048, 768, 8, "bf16")
    a = ex.exfold_workspace_bytes(qwen, 8192, 4)
    b = ex.exfold_workspace_bytes(qwen, 8192, 6)
    assert 0 < a < b
    rows = 8192 * 4
    assert a >= rows * 2048 * 2 + rows * 768 * 2 + 8192 * 2048 * 4   # sorted rows + H + fp32 accumulator
    assert a % 256 == 0
    assert ex.exfold_workspace_bytes(ex.make_layer(128, 0, 2048, 768, 8, "bf16"), 0, 4) == 0
    assert ex.exfold_workspace_bytes(ex.make_layer(1, 0, 2048, 768, 1, "bf16"), 16, 1) == 0      # N < 2
    assert ex.exfold_workspace_bytes(ex.make_layer(128, 0, 2050, 768, 8, "bf16"), 16, 1) == 0    # d % 64
    assert ex.exfold_workspace_bytes(ex.make_layer(300, 0, 2048, 768, 8, "bf16"), 16, 1) == 0    # N > 256
    assert ex.exfold_workspace_bytes(ex.make_layer(128, 0, 2048, 768, 40, "bf16"), 16, 1) == 0   # K > 32
    assert ex.exfold_host_staging_bytes(qwen, 64) >= 2 * 64 * 2048 * 2 + 64 * 128 * 4


def test_bad_arguments_are_rejected_before_launch(ex):
    layer = ex.make_layer(8, 0, 128, 256, 2, "f32")
    tabs = ex.exfold_tables(0x1000, 0x1000, 0x1000, 0x1000, None)
    p = 0x10000  # fake, aligned, never dereferenced: every call below must fail validation first
    big = 1 << 40

    def prefill(layer=layer, x=p, lg=p, T=4, wg=p, wu=p, wd=p, tables=C.byref(tabs), kp=1, y=p, ws=p, wsb=big):
        return ex.lib.exfold_moe_prefill(C.byref(layer), x, lg, T, wg, wu, wd, tables, kp, y, None, ws, wsb, None)

    def decode(layer=layer, x=p, lg=p, B=4, m=2, ws=p, wsb=big):
        return ex.lib.exfold_moe_decode(C.byref(layer), p if x else None, lg, B, p, p, p, C.byref(tabs), m, p, None,
                                        ws, wsb, None)

    assert prefill(x=None) == ex.EXFOLD_ERR_INVALID_ARG
    assert prefill(tables=None) == ex.EXFOLD_ERR_INVALID_ARG
    assert prefill(kp=0) == ex.EXFOLD_ERR_INVALID_ARG
    assert prefill(kp=3) == ex.EXFOLD_ERR_INVALID_ARG          # K' > K
    assert prefill(T=0) == ex.EXFOLD_ERR_INVALID_ARG
    assert prefill(ws=p + 8) == ex.EXFOLD_ERR_INVALID_ARG      # workspace not 256-byte aligned
    assert prefill(x=p + 4) == ex.EXFOLD_ERR_INVALID_ARG       # x not 16-byte aligned
    assert prefill(wsb=1024) == ex.EXFOLD_ERR_WORKSPACE_TOO_SMALL
    assert prefill(layer=ex.make_layer(8, 0, 128, 256, 9, "f32")) == ex.EXFOLD_ERR_INVALID_ARG  # K > N
    assert decode(m=0) == ex.EXFOLD_ERR_INVALID_ARG
    assert decode(m=9) == ex.EXFOLD_ERR_INVALID_ARG            # M > N
    assert decode(B=257) == ex.EXFOLD_ERR_UNSUPPORTED
    assert decode(wsb=1024) == ex.EXFOLD_ERR_WORKSPACE_TOO_SMALL
    opts = ex.exfold_calib_opts(1e-3, -4, 4, 1e-12, 7)
    out = ex.exfold_tables(p, p, p, p, None)
    rc = ex.lib.exfold_calibrate(C.byref(layer), p, p, 16, p, p, p, C.byref(opts), C.byref(out), p, big, None)
    assert rc == ex.EXFOLD_ERR_INVALID_ARG                     # unknown calibration mode
    assert ex.lib.exfold_device_status(None, None) == ex.EXFOLD_ERR_INVALID_ARG
    good = ex.exfold_calib_opts(1e-3, -4, 4, 1e-12, 0)
    jobs = (ex.exfold_calib_job * 2)(ex.exfold_calib_job(p, p, 16, p, p, p, C.pointer(out)),
                                     ex.exfold_calib_job(p, p, 16, p, p, p, C.pointer(out)))

    def layers(jobs=jobs, n=2, opts=good, wsb=big):
        return ex.lib.exfold_calibrate_layers(C.byref(layer), jobs, n, C.byref(opts), None, p, wsb, None)

    assert layers(n=0) == ex.EXFOLD_ERR_INVALID_ARG
    assert layers(n=257) == ex.EXFOLD_ERR_INVALID_ARG            # more jobs than EXFOLD_MAX_CALIB_JOBS
    assert layers(opts=opts) == ex.EXFOLD_ERR_INVALID_ARG        # unknown calibration mode
    assert layers(wsb=1024) == ex.EXFOLD_ERR_WORKSPACE_TOO_SMALL
    bad = (ex.exfold_calib_job * 1)(ex.exfold_calib_job(p, p, 0, p, p, p, C.pointer(out)))
    assert layers(jobs=bad, n=1) == ex.EXFOLD_ERR_INVALID_ARG    # a job without tokens

    def router(layer=layer, x=p, wr=p, T=4, lg=p, ws=p, wsb=big):
        return ex.lib.exfold_router_logits(C.byref(layer), x, wr, T, lg, ws, wsb, None)

    assert router(x=None) == ex.EXFOLD_ERR_INVALID_ARG
    assert router(wr=None) == ex.EXFOLD_ERR_INVALID_ARG
    assert router(T=0) == ex.EXFOLD_ERR_INVALID_ARG
    assert router(lg=p + 4) == ex.EXFOLD_ERR_INVALID_ARG       # logits not 16-byte aligned
    assert router(ws=p + 8) == ex.EXFOLD_ERR_INVALID_ARG
    assert router(wsb=64) == ex.EXFOLD_ERR_WORKSPACE_TOO_SMALL

    def dec_layer(wr=p, lg=p, B=4, wsb=big):
        return ex.lib.exfold_moe_decode_layer(C.byref(layer), p, wr, B, p, p, p, C.byref(tabs), 2, lg, p, None, p, wsb, None)

    def pre_layer(kp=1, T=4, wsb=big):
        return ex.lib.exfold_moe_prefill_layer(C.byref(layer), p, p, T, p, p, p, C.byref(tabs), kp, p, p, None, p, wsb, None)

    assert dec_layer(wr=None) == ex.EXFOLD_ERR_INVALID_ARG
    assert dec_layer(lg=None) == ex.EXFOLD_ERR_INVALID_ARG
    assert dec_layer(lg=p + 4) == ex.EXFOLD_ERR_INVALID_ARG    # scores buffer not 16-byte aligned
    assert dec_layer(B=0) == ex.EXFOLD_ERR_INVALID_ARG
    assert dec_layer(B=257) == ex.EXFOLD_ERR_UNSUPPORTED
    assert dec_layer(wsb=1024) == ex.EXFOLD_ERR_WORKSPACE_TOO_SMALL
    assert pre_layer(kp=3) == ex.EXFOLD_ERR_INVALID_ARG
    assert pre_layer(wsb=1024) == ex.EXFOLD_ERR_WORKSPACE_TOO_SMALL
    assert ex.lib.exfold_static_scratch_address(None) == ex.EXFOLD_ERR_INVALID_ARG


def test_product_package_does_not_touch_the_oracle():
    """The CUDA path and the oracle share no code and neither imports the other."""
    pkg = os.path.join(ROOT, "paper_2608_24938_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2608_24938_b200" not in text and "libexfold.so" not in text, f

