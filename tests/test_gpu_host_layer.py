"""The host-buffer entry points (lrbi_layer_create / _forward_host / _destroy) against the CPU oracle."""
import numpy as np
import pytest

import oracle
from paper_1905_05686_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
TOL = 5e-3


def rel_fro(got, want):
    return float(np.linalg.norm(got - want) / np.linalg.norm(want))


@pytest.mark.parametrize("batch,pinned", [(3, False), (200, True), (1500, True)])
def test_forward_from_host_memory(batch, pinned):
    from paper_1905_05686_b200 import binding as B
    L = synth.Layer("host", 384, 1024, 128, 256, 16, 0.25, 0.05)
    Ip, Iz = synth.make_factors(L)
    Wb = synth.make_weights(L)
    Xb = synth.make_activations(L, batch)
    layer = B.HostLayer(L, Wb, synth.pack_ip(Ip), synth.pack_iz(Iz), max_batch=batch)
    X = torch.from_numpy(Xb.view(np.int16)).view(torch.bfloat16)
    Y = torch.full((batch, L.rows), float("nan"), dtype=torch.bfloat16)
    if pinned:
        X, Y = X.pin_memory(), Y.pin_memory()
    want = oracle.masked_gemm(Wb, oracle.decode_mask(Ip, Iz, L.rows, L.cols), Xb)
    for _ in range(2):                                   # the handle is reusable
        layer.forward_host(X, Y)
        got = Y.float().numpy().astype(np.float64)
        assert np.isfinite(got).all() and rel_fro(got, want) <= TOL
    Y32 = torch.empty((batch, L.rows), dtype=torch.float32)
    layer.forward_host(X, Y32)
    assert rel_fro(Y32.numpy().astype(np.float64), want) <= 2e-5
    with pytest.raises(B.LrbiError):                     # more rows than the handle was created for
        layer.forward_host(torch.zeros((batch + 1, L.cols), dtype=torch.bfloat16),
                           torch.zeros((batch + 1, L.rows), dtype=torch.bfloat16))
    layer.close()
    assert B.device_status() == 0
