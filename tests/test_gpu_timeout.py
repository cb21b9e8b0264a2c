"""The timeout contract of the boundary, shown without hanging anything: a kernel whose bounded wait is
meant to run out (a barrier nobody signals, limit one millisecond) leaves its code in the status word;
the next synchronising call sees it; compute calls then refuse with LRBI_ERR_TIMEOUT until it is cleared."""
import numpy as np
import pytest

import oracle
from paper_1905_05686_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def test_a_wait_that_runs_out_is_recorded_reported_and_cleared():
    from paper_1905_05686_b200 import binding as B
    L = synth.Layer("timeout", 256, 512, 128, 256, 16, 0.25, 0.05)
    Ip, Iz = synth.make_factors(L)
    Wb, Xb = synth.make_weights(L), synth.make_activations(L, 40)
    ip, iz = B.to_device_words(synth.pack_ip(Ip)), B.to_device_words(synth.pack_iz(Iz))
    W, X = B.to_device_bf16(Wb), B.to_device_bf16(Xb)
    assert B.device_status(clear=True) in (0, 0x600)
    assert B.device_status() == 0

    B.selftest_bounded_wait(1000)
    B.lrbi_masked_gemm(L, W, ip, iz, X)                  # asynchronous: cannot know yet
    assert B.device_status() == 0x600                    # synchronises, sees the code
    assert B.lib().lrbi_last_device_error() == 0x600
    before = B.launch_count()
    for call in (lambda: B.lrbi_masked_gemm(L, W, ip, iz, X),
                 lambda: B.lrbi_decode_mask(L, ip, iz),
                 lambda: B.lrbi_masked_gemm_static(L, W, ip, iz, X, torch.empty((40, L.rows), dtype=torch.bfloat16, device="cuda"))):
        with pytest.raises(B.LrbiError) as e:
            call()
        assert e.value.code == B.ERR_TIMEOUT
    assert B.launch_count() == before                    # refused before any launch

    assert B.device_status(clear=True) == 0x600          # reports once more, then clears
    assert B.device_status() == 0
    Y = B.lrbi_masked_gemm(L, W, ip, iz, X)              # the device is usable as before
    want = oracle.masked_gemm(Wb, oracle.decode_mask(Ip, Iz, L.rows, L.cols), Xb)
    got = Y.float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - want) <= 5e-3 * np.linalg.norm(want)


def test_the_host_buffer_call_reports_a_timeout_it_can_see():
    from paper_1905_05686_b200 import binding as B
    L = synth.Layer("timeout_host", 256, 512, 128, 256, 16, 0.25, 0.05)
    Ip, Iz = synth.make_factors(L)
    layer = B.HostLayer(L, synth.make_weights(L), synth.pack_ip(Ip), synth.pack_iz(Iz), max_batch=8)
    X = torch.zeros((8, L.cols), dtype=torch.bfloat16)
    Y = torch.zeros((8, L.rows), dtype=torch.bfloat16)
    assert B.device_status(clear=True) == 0
    layer.forward_host(X, Y)
    B.selftest_bounded_wait(500)
    with pytest.raises(B.LrbiError) as e:                # this call synchronises and finds the code
        layer.forward_host(X, Y)
    assert e.value.code == B.ERR_TIMEOUT
    assert B.device_status(clear=True) == 0x600
    layer.forward_host(X, Y)
    layer.close()
    assert B.device_status() == 0
