"""The entry point for callers that may not allocate device memory.

Some users of this library run under a fixed memory budget: a server that carved up the GPU at
start-up, or a plug-in that was never given the right to call cudaMalloc (which can also block, or
fail half-way through a request).  For them lrbi_masked_gemm_static keeps the K-split partial sums in
an 8 MiB array that is part of the library itself.  This file checks, through the C ABI, that it gives
the same Y as lrbi_masked_gemm and as the CPU oracle, twice in a row (the second call finds the first
call's leftovers in the shared array), that the device's free memory does not move while it is called
again and again, and that it refuses, without launching, what does not fit.  It is collected last on
purpose, so a run that stops at the first failure has already been through every other test.
"""
import numpy as np
import pytest

import oracle
from paper_1905_05686_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

TOL = 5e-3          # same bound as the other GPU tests: relative Frobenius error


def rel_fro(got, want):
    return float(np.linalg.norm(got - want) / np.linalg.norm(want))


def _inputs(layer, batch, seed_shift=0):
    from paper_1905_05686_b200 import binding as B
    Ip, Iz = synth.make_factors(layer)
    W = B.to_device_bf16(synth.make_weights(layer))
    xl = synth.Layer(**{**layer.__dict__, "seed": layer.seed + seed_shift})
    X = B.to_device_bf16(synth.make_activations(xl, batch))
    return B, W, B.to_device_words(synth.pack_ip(Ip)), B.to_device_words(synth.pack_iz(Iz)), X


@pytest.mark.parametrize("y_dtype", ["bf16", "f32"])
def test_static_scratch_entry_point_matches_the_allocating_one_twice(y_dtype):
    layer = synth.Layer("noalloc", 1024, 4608, 512, 512, 32, 0.09, 0.01)
    batch = 16
    dt = torch.bfloat16 if y_dtype == "bf16" else torch.float32
    B, W, ip, iz, X = _inputs(layer, batch)
    need = B.masked_gemm_static_bytes(layer, batch)
    assert 0 < need <= B.STATIC_SCRATCH_BYTES, "this shape is meant to split K and to fit the fixed array"
    assert B.masked_gemm_plan(layer, batch, B.ALGO_TENSOR).k_splits > 1
    want = B.lrbi_masked_gemm(layer, W, ip, iz, X, y_dtype=dt, algo=B.ALGO_TENSOR).float().cpu().numpy().astype(np.float64)
    Ip, Iz = synth.make_factors(layer)
    ref = oracle.masked_gemm(synth.make_weights(layer), oracle.decode_mask(Ip, Iz, layer.rows, layer.cols),
                             synth.make_activations(layer, batch))
    assert rel_fro(want, ref) <= (TOL if y_dtype == "bf16" else 2e-5)
    for call in range(2):
        # a different batch in between leaves other partial sums behind in the shared array
        if call == 1:
            _, _, _, _, X2 = _inputs(layer, 24, seed_shift=7)
            B.lrbi_masked_gemm_static(layer, W, ip, iz, X2, torch.empty((24, layer.rows), dtype=dt, device="cuda"))
        Y = torch.full((batch, layer.rows), float("nan"), dtype=dt, device="cuda")
        B.lrbi_masked_gemm_static(layer, W, ip, iz, X, Y)
        torch.cuda.synchronize()
        got = Y.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert rel_fro(got, want) <= TOL, (call, rel_fro(got, want))
        assert rel_fro(got, ref) <= (TOL if y_dtype == "bf16" else 2e-5), (call, rel_fro(got, ref))
    assert B.device_status() == 0


def test_static_scratch_entry_point_leaves_free_memory_alone():
    """After one warm-up call (module load, address look-up) the driver's count of free device bytes does
    not move, however often the entry point is called and whatever batch it is given."""
    layer = synth.Layer("noalloc", 1024, 4608, 512, 512, 32, 0.09, 0.01)
    B, W, ip, iz, X16 = _inputs(layer, 16)
    _, _, _, _, X48 = _inputs(layer, 48, seed_shift=3)
    Y16 = torch.empty((16, layer.rows), dtype=torch.bfloat16, device="cuda")
    Y48 = torch.empty((48, layer.rows), dtype=torch.float32, device="cuda")
    B.lrbi_masked_gemm_static(layer, W, ip, iz, X16, Y16)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(20):
        B.lrbi_masked_gemm_static(layer, W, ip, iz, X16, Y16)
        B.lrbi_masked_gemm_static(layer, W, ip, iz, X48, Y48)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)


def test_static_scratch_entry_point_needs_no_scratch_for_large_batches():
    layer = synth.Layer("noalloc_big", 512, 1024, 128, 256, 16, 0.3, 0.02)
    batch = 40 * 256                 # 40 batch tiles x 4 row blocks: enough tiles, K is not split
    B, W, ip, iz, X = _inputs(layer, batch)
    assert B.masked_gemm_static_bytes(layer, batch) == 0
    want = B.lrbi_masked_gemm(layer, W, ip, iz, X, algo=B.ALGO_TENSOR).float().cpu().numpy().astype(np.float64)
    Y = torch.empty((batch, layer.rows), dtype=torch.bfloat16, device="cuda")
    B.lrbi_masked_gemm_static(layer, W, ip, iz, X, Y)
    got = Y.float().cpu().numpy().astype(np.float64)
    assert rel_fro(got, want) <= TOL
    Ip, Iz = synth.make_factors(layer)
    ref = oracle.masked_gemm(synth.make_weights(layer), oracle.decode_mask(Ip, Iz, layer.rows, layer.cols),
                             synth.make_activations(layer, batch))
    assert rel_fro(got, ref) <= TOL


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    layer = synth.CONFIGS["alexnet_fc"]
    batch = 128                      # 10 splits x 128 x 4096 fp32 = 21 MB of partial sums
    from paper_1905_05686_b200 import binding as B
    assert B.masked_gemm_static_bytes(layer, batch) > B.STATIC_SCRATCH_BYTES
    B2, W, ip, iz, X = _inputs(layer, batch)
    Y = torch.zeros((batch, layer.rows), dtype=torch.bfloat16, device="cuda")
    before = B.launch_count()
    with pytest.raises(B.LrbiError) as e:
        B.lrbi_masked_gemm_static(layer, W, ip, iz, X, Y)
    assert e.value.code == B.ERR_TOO_LARGE
    assert B.launch_count() == before and not Y.any()
