"""The allocation-free decode entry point against the ordinary one.

exfold_moe_decode_noalloc exists for hosts that may not allocate device memory while they run (a
fixed start-up memory pool, a plugin without an allocator of its own): its scratch is a fixed
array inside the library. This file is collected last on purpose, so a run that stops at the
first failure has already been through every other test. It passes alone in a fresh process and
after the rest of the suite.
"""
import numpy as np
import pytest
import torch

import synth_inputs as si
from harness import Case, check_output

pytestmark = pytest.mark.gpu


def test_noalloc_decode_matches_workspace_decode_twice_in_a_row():
    cfg = si.LayerConfig("noalloc", 16, 1, 256, 384, 4, "bf16", 64, (2,), 24, (6,), logits="zipf")
    case = Case(cfg)
    ex, dev = case.ex, case.dev
    M, B, K, N = 6, case.B, cfg.top_k, cfg.n_experts
    ref = case.run_decode(M)                      # existing entry point, caller-provided workspace
    orc = case.oracle_decode(M)                   # and the CPU oracle, independently of both
    scale = np.abs(ref["y"]).max()
    ys = [torch.full((B, cfg.hidden), float("nan"), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    metas = [dict(ids=torch.full((B, K), -7, dtype=torch.int32, device=dev),
                  w=torch.full((B, K), float("nan"), dtype=torch.float32, device=dev),
                  pool_ids=torch.full((M,), -7, dtype=torch.int32, device=dev)) for _ in range(2)]
    torch.cuda.synchronize()
    for call in range(2):                         # the shared array keeps the previous call's contents
        y, meta = ys[call], metas[call]
        # everything the call touches exists already: from here to the end of the call nothing may be allocated
        torch_before = torch.cuda.memory_allocated(dev)
        free_before, _ = torch.cuda.mem_get_info(dev)
        ex.exfold_moe_decode_noalloc(case.layer, case.d_xd, case.d_lgd, case.d_wg, case.d_wu, case.d_wd,
                                     case.tables, M, y, meta=meta)
        assert ex.exfold_device_status_noalloc() == ex.EXFOLD_OK    # synchronises; no bounded wait ran out
        if call == 1:   # (the first call on a device may still load the library's kernels, which takes device memory)
            assert torch.cuda.memory_allocated(dev) == torch_before
            assert torch.cuda.mem_get_info(dev)[0] == free_before, "device memory was allocated during the call"
        got = y.float().cpu().numpy()
        assert np.isfinite(got).all(), f"call {call}: output not fully written"
        assert np.array_equal(meta["ids"].cpu().numpy(), ref["ids"])
        assert np.array_equal(meta["pool_ids"].cpu().numpy(), ref["pool_ids"])
        assert np.array_equal(meta["w"].cpu().numpy(), ref["w"])
        # same tolerance as the parity tests use for bf16 outputs
        assert np.abs(got - ref["y"]).max() <= 2e-2 * scale
        assert np.linalg.norm(got - ref["y"]) <= 1e-2 * np.linalg.norm(ref["y"])
        # against the oracle: integers bit for bit, outputs within the parity tolerance
        assert np.array_equal(meta["ids"].cpu().numpy(), orc["ids"])
        assert np.array_equal(meta["pool_ids"].cpu().numpy(), orc["pool_ids"][:M])
        check_output(got, orc["y"], "bf16")


def test_noalloc_status_record_is_read_and_cleared():
    """The status record of the allocation-free calls sits in the library's own array, where exfold_device_status
    cannot be pointed; exfold_device_status_noalloc reads it. A code is written there from the host (no kernel is
    made to time out), reported once and cleared; a stale code does not survive the next call."""
    from paper_2608_24938_b200 import binding as ex
    import ctypes as C
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    addr = ex.exfold_static_scratch_address()
    assert addr != 0 and addr % 256 == 0
    assert ex.exfold_static_scratch_address() == addr        # looked up once per device
    rt = C.CDLL("libcudart.so.12")   # the runtime torch has already loaded
    rt.cudaMemcpy.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_int]

    def poke(code):
        src = C.c_int32(code)
        assert rt.cudaMemcpy(addr, C.byref(src), 4, 1) == 0   # host -> device
        torch.cuda.synchronize()

    poke(0)
    assert ex.exfold_device_status_noalloc() == ex.EXFOLD_OK
    poke(ex.EXFOLD_ERR_DEVICE_TIMEOUT)
    assert ex.exfold_device_status_noalloc() == ex.EXFOLD_ERR_DEVICE_TIMEOUT
    assert ex.exfold_device_status_noalloc() == ex.EXFOLD_OK
    poke(-77)
    assert ex.exfold_device_status_noalloc() == ex.EXFOLD_ERR_CUDA
    poke(ex.EXFOLD_ERR_DEVICE_TIMEOUT)
    cfg = si.LayerConfig("noalloc", 16, 1, 256, 384, 4, "bf16", 64, (2,), 24, (6,), logits="zipf")
    case = Case(cfg)
    y = torch.empty((case.B, cfg.hidden), dtype=torch.bfloat16, device=dev)
    ex.exfold_moe_decode_noalloc(case.layer, case.d_xd, case.d_lgd, case.d_wg, case.d_wu, case.d_wd, case.tables, 6, y)
    assert ex.exfold_device_status_noalloc() == ex.EXFOLD_OK


def test_noalloc_decode_rejects_what_does_not_fit():
    cfg = si.LayerConfig("noalloc-big", 16, 0, 2048, 4096, 4, "bf16", 64, (2,), 256, (6,))
    from paper_2608_24938_b200 import binding as ex
    dev = torch.device("cuda:0")
    layer = ex.make_layer(16, 0, 2048, 4096, 4, "bf16")
    assert ex.exfold_workspace_bytes(layer, 256, 4) > ex.EXFOLD_STATIC_SCRATCH_BYTES
    small = torch.zeros(4096, dtype=torch.float32, device=dev)  # never read: the size check comes first
    tabs = ex.make_tables(small, small, small, small)
    xfake = torch.zeros((256, 8), dtype=torch.bfloat16, device=dev)
    before = ex.exfold_launch_count()
    rc = ex.exfold_moe_decode_noalloc(layer, xfake, small, small, small, small, tabs, 4, xfake, check=False)
    assert rc == ex.EXFOLD_ERR_EXCEEDS_STATIC_SCRATCH
    assert "EXFOLD_STATIC_SCRATCH_BYTES" in ex.exfold_status_string(rc)
    assert ex.exfold_launch_count() == before
