"""The bounded device-side waits, exercised without a fault: a manifest built with
GMS_BUILD_SELFTEST_STALL tells one barrier to expect 16 bytes that are never sent, so the warp that
waits on it runs into its 2-second limit, raises GMS_DEV_TIMEOUT in the status word, drains what it
has in flight and returns while every other warp finishes.  The context must stay usable: the same
image restored right afterwards through a normal manifest matches the oracle bit for bit."""
import time

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402

from gpu_harness import FILL, DeviceWorkload, oracle_record  # noqa: E402


@pytest.mark.parametrize("call", ["restore", "digest"])
def test_a_wait_that_runs_out_sets_the_status_bit_and_leaves_the_context_usable(oracle, call):
    w = W.mixed_manifest(n_small=400, n_large=1, large_bytes=2 << 20)
    image = W.random_bytes_host(w.image_bytes, seed=77)
    d = DeviceWorkload(w, image)
    stalled = gms.gms_manifest_build(d.entries, w.image_bytes, flags=gms.BUILD_SELFTEST_STALL)

    t0 = time.perf_counter()
    if call == "restore":
        gms.gms_restore(stalled, d.image, gms.SRC_DEVICE, d.bd_ptr(), d.td_ptr())
    else:
        gms.gms_digest(stalled, d.bd_ptr(), d.td_ptr())
    torch.cuda.synchronize()  # returns: the kernel ended by itself
    waited = time.perf_counter() - t0
    assert 1.5 < waited < 30.0, waited  # one wait limit for the stalled block, one more while draining it
    with pytest.raises(gms.GmsError) as ei:  # the status call turns the bit into GMS_ERR_TIMEOUT
        gms.gms_last_device_status(stalled)
    assert ei.value.status == gms.ERR_TIMEOUT
    stalled.close()

    # same process, same context, same buffers: a normal restore is exact
    want_slab = np.full(w.slab_bytes, FILL, np.uint8)
    rc, want_bd, want_td = oracle.restore(oracle_record(oracle, w), image, want_slab)
    assert rc == 0
    bd, td = d.restore()
    assert np.array_equal(d.slab_host(), want_slab)
    assert np.array_equal(bd, want_bd) and np.array_equal(td, want_td)
    d.close()
