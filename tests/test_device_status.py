"""The bounded waits of the kernels and their error path, exercised without harming the device:
a wait that nothing ever satisfies runs out after a few milliseconds, the kernel returns
normally, the status word names the wait, and the next ordinary call is unaffected."""
import numpy as np
import pytest
import torch

from paper_2505_18663_b200 import binding as B
from paper_2505_18663_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def small_layer():
    wl = W.WORKLOADS["tiny"]
    layer = wl.layers[0]
    x = W.make_activations(wl, layer.K, device=DEV)
    u, d, z = W.make_weight_codes(layer, seed=0, device=DEV)
    blob = torch.empty(B.dvdq_weight_blob_bytes(layer.N, layer.K), dtype=torch.uint8, device=DEV)
    w = B.dvdq_pack_weights(u, d, z, layer.rot_block, blob)
    q = B.ActQuant(layer.bits, layer.rot_block, 0, 8)
    ws = torch.empty(B.dvdq_qlinear_workspace_bytes(wl.M, layer.K, q), dtype=torch.uint8, device=DEV)
    Y = torch.empty(wl.M, layer.N, dtype=torch.bfloat16, device=DEV)

    def run():
        B.dvdq_qlinear(x, q, w, None, 0, Y, ws)
        return Y.clone()
    return run, blob


def test_a_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    run, _keep = small_layer()
    before = run()
    assert B.dvdq_last_device_status() == (B.OK, 0)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    B.dvdq_debug_wait_timeout(3_000_000)                        # 3 ms
    t1.record()
    status, detail = B.dvdq_last_device_status()                # synchronizes
    assert status == B.ERR_DEVICE_TIMEOUT and detail == 8       # the debug wait's id
    ms = t0.elapsed_time(t1)
    assert 3.0 <= ms < 500.0, ms                                # it waited for the limit, and not much longer
    # reading the word clears it; the next ordinary call runs and gives the same bits as before
    assert B.dvdq_last_device_status() == (B.OK, 0)
    after = run()
    assert torch.equal(before, after)
    assert B.dvdq_last_device_status() == (B.OK, 0)


def test_wait_limit_is_validated():
    with pytest.raises(B.DvdqError) as e:
        B.dvdq_debug_wait_timeout(0)
    assert e.value.status == B.ERR_SHAPE
    with pytest.raises(B.DvdqError) as e:
        B.dvdq_debug_wait_timeout(5_000_000_000)
    assert e.value.status == B.ERR_SHAPE


def test_int8_ceiling_runs_and_reports_its_work():
    ops = B.dvdq_int8_mma_ceiling(2000)
    torch.cuda.synchronize()
    props = torch.cuda.get_device_properties(0)
    pairs = props.multi_processor_count // 2
    assert ops == pairs * 2000 * 4 * 2 * 256 * 256 * 32
    assert B.dvdq_last_device_status() == (B.OK, 0)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    ops = B.dvdq_int8_mma_ceiling(20000)
    t1.record()
    torch.cuda.synchronize()
    tops = ops / (t0.elapsed_time(t1) * 1e-3) / 1e12
    # an issue loop on resident operands cannot beat the nominal dense int8 rate, and a healthy one is far above half of it
    assert 2000.0 < tops < 4700.0, tops
    with pytest.raises(B.DvdqError):
        B.dvdq_int8_mma_ceiling(0)


def test_two_host_threads_share_the_library():
    """The launch-time set-up is cached per device under a lock: two host threads that call the
    library at the same time (own streams, own buffers) get the bits a single thread gets."""
    import threading
    wl = W.WORKLOADS["tiny"]
    layer = wl.layers[0]
    x = W.make_activations(wl, layer.K, device=DEV)
    u, d, z = W.make_weight_codes(layer, seed=0, device=DEV)
    blob = torch.empty(B.dvdq_weight_blob_bytes(layer.N, layer.K), dtype=torch.uint8, device=DEV)
    w = B.dvdq_pack_weights(u, d, z, layer.rot_block, blob)
    torch.cuda.synchronize()
    results, errors = {}, []

    def worker(idx, container):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            q = B.ActQuant(layer.bits, layer.rot_block, 0, container)
            ws = torch.empty(B.dvdq_qlinear_workspace_bytes(wl.M, layer.K, q), dtype=torch.uint8, device=DEV)
            Y = torch.empty(wl.M, layer.N, dtype=torch.bfloat16, device=DEV)
            for _ in range(20):
                B.dvdq_qlinear(x, q, w, None, 0, Y, ws, stream=stream)
            stream.synchronize()
            results[idx] = Y
        except Exception as e:   # surfaced by the assertion below
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(i, 8 if i % 2 else 0)) for i in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert B.dvdq_last_device_status() == (B.OK, 0)
    # both layouts give the same output; every thread got it
    for i in range(1, 4):
        assert torch.equal(results[0], results[i])
