"""More parity cases on the GPU: every compiled ring depth and several warp counts / claim modes
(each in a process of its own, since the launch shape is fixed once per process), image base
addresses that are only 16-byte aligned, calls on a non-default stream, and two manifests
restored concurrently on two streams."""
import os
import subprocess
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402

from gpu_harness import FILL, DeviceWorkload, oracle_record  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))

SHAPES = [
    {"GMS_GEOM_RESTORE": "4,3,1", "GMS_GEOM_DIGEST": "4,3,1", "GMS_GEOM_KV": "4,3,1"},
    {"GMS_GEOM_RESTORE": "12,4,1", "GMS_GEOM_DIGEST": "12,4,1", "GMS_GEOM_KV": "12,4,1", "GMS_CHUNK_BLOCKS": "1"},
    {"GMS_GEOM_RESTORE": "6,8,1", "GMS_GEOM_DIGEST": "6,8,1", "GMS_GEOM_KV": "6,8,1", "GMS_CHUNK_BLOCKS": "32"},
    {"GMS_GEOM_RESTORE": "6,4,2", "GMS_GEOM_DIGEST": "8,3,2", "GMS_GEOM_KV": "4,6,2", "GMS_CLAIM_RESTORE": "8,3",
     "GMS_CLAIM_DIGEST": "1,1", "GMS_CHUNK_BLOCKS": "7", "GMS_CHUNK_BLOCKS_DIGEST": "2"},
    {"GMS_GEOM_RESTORE": "16,3,1", "GMS_CLAIM_RESTORE": "32,2", "GMS_CLAIM_DIGEST": "32,64", "GMS_CHUNK_BLOCKS_DIGEST": "32"},
    {"GMS_L2_KEEP": "1"},  # the digest-only kernels' L2 hints, which small cases would not get by themselves
    {"GMS_L2_KEEP": "1", "GMS_GEOM_DIGEST": "12,4,1", "GMS_CHUNK_BLOCKS_DIGEST": "3"},
]


@pytest.mark.parametrize("env", SHAPES, ids=lambda e: " ".join(f"{k[4:]}={v}" for k, v in e.items()))
def test_parity_in_other_launch_shapes(env):
    full = dict(os.environ)
    full.update(env)
    full["GMS_TUNING_HOOKS"] = "1"  # the library ignores the shape hooks without it
    full["GMS_CHECK_TABLES"] = "1"  # every manifest built in the child compares its device-written work lists with the host's
    r = subprocess.run([sys.executable, os.path.join(HERE, "geometry_check.py")], env=full, capture_output=True, text=True,
                       timeout=600)
    assert r.returncode == 0 and r.stdout.strip().startswith("OK"), r.stdout[-2000:] + r.stderr[-4000:]


def test_short_randomised_soak():
    """Ten seconds of tests/fuzz_parity.py (random manifests, operations, corruption, KV lists) against the oracle."""
    r = subprocess.run([sys.executable, os.path.join(HERE, "fuzz_parity.py"), "--seconds", "10", "--seed", "7"],
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "FUZZ OK" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


def test_image_base_only_16_byte_aligned(oracle):
    w = W.mixed_manifest(n_small=700, n_large=1, large_bytes=(3 << 20) + 8, round16=False, seed=55)
    image = W.random_bytes_host(w.image_bytes, seed=6)
    slab_h = np.full(w.slab_bytes, FILL, np.uint8)
    rc, obd, otd = oracle.restore(oracle_record(oracle, w), image, slab_h)
    for shift in (16, 4080, 240):
        buf = torch.zeros(w.image_bytes + 8192, dtype=torch.uint8, device="cuda")
        buf[shift:shift + w.image_bytes] = torch.from_numpy(image).cuda()
        d = DeviceWorkload(w, image_dev=buf)
        bd, td = d.restore(image=buf.data_ptr() + shift)
        assert np.array_equal(d.slab_host(), slab_h) and np.array_equal(bd, obd) and np.array_equal(td, otd), shift
        d.close()


def test_calls_on_a_side_stream_and_two_manifests_concurrently(oracle):
    ws = [W.mixed_manifest(n_small=900, n_large=2, large_bytes=(6 << 20) + 40, round16=False, seed=s) for s in (71, 72)]
    images = [W.random_bytes_host(w.image_bytes, seed=80 + i) for i, w in enumerate(ws)]
    wants = []
    for w, img in zip(ws, images):
        slab_h = np.full(w.slab_bytes, FILL, np.uint8)
        rc, obd, otd = oracle.restore(oracle_record(oracle, w), img, slab_h)
        wants.append((slab_h, obd, otd))
    ds = [DeviceWorkload(w, img) for w, img in zip(ws, images)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for rep in range(3):
        for d in ds:
            d.slab.fill_(FILL)
            d.reset_outputs()
        torch.cuda.synchronize()
        # each manifest has its own work counters and status word, so the two restores may overlap on the GPU
        for d, s in zip(ds, streams):
            gms.gms_restore(d.m, d.image, gms.SRC_DEVICE, d.bd_ptr(), d.td_ptr(), stream=s)
            gms.gms_digest(d.m, d.bd_ptr(), d.td_ptr(), stream=s)
        for s in streams:
            s.synchronize()
        from gpu_harness import payload_of

        for d, (slab_h, obd, otd) in zip(ds, wants):
            assert np.array_equal(d.slab_host(), slab_h)
            assert np.array_equal(payload_of(d.bd, d.nb), obd) and np.array_equal(payload_of(d.td, d.nt), otd)
            assert gms.gms_last_device_status(d.m) == 0
    for d in ds:
        d.close()
