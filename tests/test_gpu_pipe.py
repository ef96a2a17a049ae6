"""gms_restore_fd: restore fed from a file through a ring of pinned buffers and the copy engine.  The
result must be exactly what gms_restore produces from the same bytes, so the oracle's restore of the
file's contents is the reference: destination bytes, block digests, tensor digests, bit-exact -- with
buffers far smaller than the tensors (tensors span many windows), file offsets that are 4 KiB-aligned
(windows read with O_DIRECT where the file system takes it), 16-byte-aligned and odd, odd sizes, and
the error paths (short file, bad arguments).  gms_capture_fd, the way back, must leave in the file exactly what the
oracle's capture leaves in an image: every tensor's bytes in place, every byte between them as it was."""
import ctypes
import os

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2609_25451_b200 import gms  # noqa: E402
from paper_2609_25451_b200 import workloads as W  # noqa: E402

from gpu_harness import FILL, DeviceWorkload, oracle_record  # noqa: E402


def test_pipe_argument_checks_need_no_gpu():
    out = ctypes.c_void_p()
    L = gms.lib()
    assert L.gms_pipe_create(1, 1 << 20, 4, ctypes.byref(out)) == gms.ERR_ARG      # fewer than 2 buffers
    assert L.gms_pipe_create(2, 4096, 4, ctypes.byref(out)) == gms.ERR_ARG          # buffer below 1 MiB
    assert L.gms_pipe_create(2, (1 << 20) + 8, 4, ctypes.byref(out)) == gms.ERR_ARG  # not a multiple of 4096
    assert L.gms_pipe_create(2, 1 << 20, 0, ctypes.byref(out)) == gms.ERR_ARG       # no readers
    assert L.gms_pipe_create(2, 1 << 20, 4, None) == gms.ERR_NULL
    assert L.gms_pipe_destroy(None) == gms.OK
    assert L.gms_pipe_direct_io(None, 1) == gms.ERR_NULL
    assert L.gms_pipe_mapped_writes(None, 1) == gms.ERR_NULL
    assert L.gms_restore_fd(None, None, 0, 0, None, None, None, None) == gms.ERR_NULL
    assert L.gms_capture_fd(None, None, 0, 0, None, None, None, None) == gms.ERR_NULL
    assert "file" in gms.gms_strerror(gms.ERR_IO)


def _write_image(path, image: np.ndarray, file_offset: int):
    with open(path, "wb") as f:
        f.write(b"\xAB" * file_offset)
        f.write(image.tobytes())


@pytest.mark.gpu
@pytest.mark.parametrize("n_buffers,buffer_mib,n_readers,file_offset",
                         [(2, 1, 1, 0), (3, 2, 4, 4096 + 16), (4, 16, 8, 512), (3, 4, 6, 8192), (2, 2, 3, 5)])
def test_restore_fd_equals_restore_of_the_same_bytes(oracle, tmp_path, n_buffers, buffer_mib, n_readers, file_offset):
    w = W.mixed_manifest(n_small=1500, n_large=3, large_bytes=(7 << 20) + 40, round16=False, seed=123)
    image = W.random_bytes_host(w.image_bytes, seed=77)
    slab_h = np.full(w.slab_bytes, FILL, np.uint8)
    rc, obd, otd = oracle.restore(oracle_record(oracle, w), image, slab_h)
    assert rc == 0
    path = str(tmp_path / "image.bin")
    _write_image(path, image, file_offset)
    d = DeviceWorkload(w, image_dev=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    pipe = gms.gms_pipe_create(n_buffers, buffer_mib << 20, n_readers)
    fd = os.open(path, os.O_RDONLY)
    try:
        for direct in (False, True):  # twice: the second call must not be disturbed by what the first left in the buffers
            gms.gms_pipe_direct_io(pipe, direct)  # second pass: O_DIRECT reads where the file system takes them
            d.slab.fill_(FILL)
            d.reset_outputs()
            st = gms.gms_restore_fd(d.m, pipe, fd, file_offset, d.bd_ptr(), d.td_ptr())
            assert gms.gms_last_device_status(d.m) == 0
            from gpu_harness import payload_of

            assert np.array_equal(d.slab_host(), slab_h), "destination bytes (or guard bands) differ"
            assert np.array_equal(payload_of(d.bd, d.nb), obd) and np.array_equal(payload_of(d.td, d.nt), otd)
            assert st["windows"] >= w.image_bytes // (buffer_mib << 20) and st["bytes_read"] <= w.image_bytes
            # windows go through the copy engine; whether reads bypass the page cache is up to the file system
            assert st["copy_engine"] == 1 and st["direct_io"] in ((0, 1) if direct else (0,))
    finally:
        os.close(fd)
        pipe.close()
        d.close()


@pytest.mark.gpu
@pytest.mark.parametrize("n_buffers,buffer_mib", [(2, 1), (3, 4), (4, 32)])
def test_restore_staged_equals_restore_of_the_same_bytes(oracle, n_buffers, buffer_mib):
    """Copy-engine-fed variant: pinned host image -> device ring -> restore kernel, ordered by stream events only."""
    from gpu_harness import payload_of

    w = W.mixed_manifest(n_small=1500, n_large=3, large_bytes=(7 << 20) + 40, round16=False, seed=321)
    image = W.random_bytes_host(w.image_bytes, seed=78)
    slab_h = np.full(w.slab_bytes, FILL, np.uint8)
    rc, obd, otd = oracle.restore(oracle_record(oracle, w), image, slab_h)
    assert rc == 0
    hptr, _, arr = gms.gms_host_image_alloc(w.image_bytes)
    arr[:] = image
    d = DeviceWorkload(w, image_dev=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    stage = gms.gms_stage_create(n_buffers, buffer_mib << 20)
    try:
        for _ in range(3):  # back to back: the ring and its events carry over from call to call
            d.slab.fill_(FILL)
            d.reset_outputs()
            gms.gms_restore_staged(d.m, stage, hptr, d.bd_ptr(), d.td_ptr())
            torch.cuda.synchronize()
            assert gms.gms_last_device_status(d.m) == 0
            assert np.array_equal(d.slab_host(), slab_h), "destination bytes (or guard bands) differ"
            assert np.array_equal(payload_of(d.bd, d.nb), obd) and np.array_equal(payload_of(d.td, d.nt), otd)
        # the source must be pinned host memory
        with pytest.raises(gms.GmsError) as ei:
            gms.gms_restore_staged(d.m, stage, d.slab, None, None)
        assert ei.value.status == gms.ERR_KIND
    finally:
        torch.cuda.synchronize()
        stage.close()
        d.close()
        gms.gms_host_image_free(hptr)


@pytest.mark.gpu
def test_piecewise_restores_with_tensors_that_share_image_bytes(oracle, tmp_path):
    """Overlapping sources are legal for a restore (several tensors filled from the same image bytes).  The window
    plan then has to sort chunks of different tensors among each other; both piecewise restores must still give the
    oracle's bytes and digests."""
    from gpu_harness import payload_of

    w = W.pack_layout("shared", [(3 << 20) + 40, 70000, 5 << 20, 4096, 1 << 20], seed=9)
    w.rows["src_offset"][2] = w.rows["src_offset"][0] + 65536   # tensor 2 starts inside tensor 0 and runs past its end
    w.rows["src_offset"][3] = w.rows["src_offset"][1]           # tensor 3 is the head of tensor 1
    image = W.random_bytes_host(w.image_bytes, seed=79)
    slab_h = np.full(w.slab_bytes, FILL, np.uint8)
    rc, obd, otd = oracle.restore(oracle_record(oracle, w), image, slab_h)
    assert rc == 0
    d = DeviceWorkload(w, image_dev=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    hptr, _, arr = gms.gms_host_image_alloc(w.image_bytes)
    arr[:] = image
    path = str(tmp_path / "shared.bin")
    _write_image(path, image, 0)
    stage = gms.gms_stage_create(2, 1 << 20)
    pipe = gms.gms_pipe_create(2, 1 << 20, 3)
    fd = os.open(path, os.O_RDONLY)
    try:
        for how in ("staged", "fd", "staged"):
            d.slab.fill_(FILL)
            d.reset_outputs()
            if how == "staged":
                gms.gms_restore_staged(d.m, stage, hptr, d.bd_ptr(), d.td_ptr())
            else:
                gms.gms_restore_fd(d.m, pipe, fd, 0, d.bd_ptr(), d.td_ptr())
            torch.cuda.synchronize()
            assert gms.gms_last_device_status(d.m) == 0
            assert np.array_equal(d.slab_host(), slab_h), how
            assert np.array_equal(payload_of(d.bd, d.nb), obd) and np.array_equal(payload_of(d.td, d.nt), otd), how
    finally:
        os.close(fd)
        torch.cuda.synchronize()
        pipe.close()
        stage.close()
        d.close()
        gms.gms_host_image_free(hptr)


def test_stage_argument_checks_need_no_gpu():
    out = ctypes.c_void_p()
    L = gms.lib()
    assert L.gms_stage_create(1, 1 << 20, ctypes.byref(out)) == gms.ERR_ARG
    assert L.gms_stage_create(2, 1000, ctypes.byref(out)) == gms.ERR_ARG
    assert L.gms_stage_create(2, 1 << 20, None) == gms.ERR_NULL
    assert L.gms_stage_destroy(None) == gms.OK
    assert L.gms_restore_staged(None, None, None, None, None, None) == gms.ERR_NULL


@pytest.mark.gpu
def test_restore_fd_reports_a_short_file(tmp_path):
    w = W.pack_layout("short", [3 << 20, 5 << 20, 100], seed=5)
    image = W.random_bytes_host(w.image_bytes, seed=1)
    path = str(tmp_path / "short.bin")
    _write_image(path, image[: w.image_bytes - (2 << 20)], 0)  # the file ends 2 MiB early
    d = DeviceWorkload(w, image_dev=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    pipe = gms.gms_pipe_create(2, 1 << 20, 2)
    fd = os.open(path, os.O_RDONLY)
    try:
        with pytest.raises(gms.GmsError) as ei:
            gms.gms_restore_fd(d.m, pipe, fd, 0, None, None)
        assert ei.value.status == gms.ERR_IO
        # the pipe and the manifest remain usable after the error
        os.close(fd)
        _write_image(path, image, 0)
        fd = os.open(path, os.O_RDONLY)
        gms.gms_restore_fd(d.m, pipe, fd, 0, None, None)
        for r in w.rows:
            s, o, n = int(r["src_offset"]), int(r["dst_offset"]), int(r["nbytes"])
            assert np.array_equal(d.slab[o:o + n].cpu().numpy(), image[s:s + n])
    finally:
        os.close(fd)
        pipe.close()
        d.close()


@pytest.mark.gpu
def test_restore_fd_empty_manifest(tmp_path):
    w = W.pack_layout("empty", [0, 0], seed=1)
    path = str(tmp_path / "e.bin")
    _write_image(path, np.zeros(16, np.uint8), 0)
    d = DeviceWorkload(w, image_dev=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    pipe = gms.gms_pipe_create(2, 1 << 20, 1)
    fd = os.open(path, os.O_RDONLY)
    try:
        d.reset_outputs()
        st = gms.gms_restore_fd(d.m, pipe, fd, 0, d.bd_ptr(), d.td_ptr())
        from gpu_harness import payload_of

        assert st["windows"] == 0 and (payload_of(d.td, d.nt) == 0).all()
    finally:
        os.close(fd)
        pipe.close()
        d.close()


PATTERN = 0xA5  # what the file holds before a capture


@pytest.mark.gpu
@pytest.mark.parametrize("n_buffers,buffer_mib,n_writers,file_offset",
                         [(2, 1, 1, 0), (3, 2, 4, 4096 + 16), (4, 16, 8, 5), (2, 4, 3, 8192)])
def test_capture_fd_leaves_in_the_file_what_the_oracle_captures(oracle, tmp_path, n_buffers, buffer_mib, n_writers, file_offset):
    from gpu_harness import payload_of

    w = W.mixed_manifest(n_small=1500, n_large=3, large_bytes=(7 << 20) + 40, round16=False, seed=124)
    tail = 100  # bytes of the file behind the image: must stay untouched as well
    path = str(tmp_path / "snapshot.bin")
    d = DeviceWorkload(w, image_dev=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    pipe = gms.gms_pipe_create(n_buffers, buffer_mib << 20, n_writers)
    try:
        for seed in (31, 32):  # twice with different contents: nothing of the first pass may show in the second file
            slab_h = W.random_bytes_host(w.slab_bytes, seed=seed)
            d.slab.copy_(torch.from_numpy(slab_h))
            want = np.full(w.image_bytes, PATTERN, np.uint8)
            rc, obd, otd = oracle.capture(oracle_record(oracle, w), want, slab_h)
            assert rc == 0
            with open(path, "wb") as f:
                f.write(bytes([PATTERN]) * (file_offset + w.image_bytes + tail))
            # second pass: the writers store through a shared mapping of the file (needs a descriptor that may be mapped)
            mapped = seed == 32
            gms.gms_pipe_mapped_writes(pipe, mapped)
            fd = os.open(path, os.O_RDWR if mapped else os.O_WRONLY)
            try:
                d.reset_outputs()
                st = gms.gms_capture_fd(d.m, pipe, fd, file_offset, d.bd_ptr(), d.td_ptr())
            finally:
                os.close(fd)
            assert gms.gms_last_device_status(d.m) == 0 and st["mapped_io"] == (1 if mapped else 0)
            got = np.fromfile(path, dtype=np.uint8)
            assert got.size == file_offset + w.image_bytes + tail, "the file's length changed"
            assert (got[:file_offset] == PATTERN).all() and (got[file_offset + w.image_bytes:] == PATTERN).all()
            assert np.array_equal(got[file_offset:file_offset + w.image_bytes], want), "tensor bytes or the gaps between them differ"
            assert np.array_equal(payload_of(d.bd, d.nb), obd) and np.array_equal(payload_of(d.td, d.nt), otd)
            assert np.array_equal(d.slab_host(), slab_h), "capture wrote to the allocations"
            assert st["bytes_read"] == sum(int(r["nbytes"]) for r in w.rows)
            assert st["windows"] >= w.image_bytes // (buffer_mib << 20)
        # and back: a restore fed from that file reproduces the allocations it was captured from
        d.slab.fill_(FILL)
        fd = os.open(path, os.O_RDONLY)
        try:
            d.reset_outputs()
            gms.gms_restore_fd(d.m, pipe, fd, file_offset, d.bd_ptr(), d.td_ptr())
        finally:
            os.close(fd)
        assert np.array_equal(payload_of(d.bd, d.nb), obd) and np.array_equal(payload_of(d.td, d.nt), otd)
        back = d.slab_host()
        for r in w.rows:
            o, n = int(r["dst_offset"]), int(r["nbytes"])
            assert np.array_equal(back[o:o + n], slab_h[o:o + n])
    finally:
        pipe.close()
        d.close()


@pytest.mark.gpu
def test_capture_fd_error_paths(tmp_path):
    w = W.pack_layout("cap-err", [3 << 20, 0, 100], seed=6)
    d = DeviceWorkload(w, image_dev=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    d.slab.copy_(torch.from_numpy(W.random_bytes_host(w.slab_bytes, seed=9)))
    pipe = gms.gms_pipe_create(2, 1 << 20, 2)
    path = str(tmp_path / "ro.bin")
    with open(path, "wb") as f:
        f.write(b"\0" * w.image_bytes)
    fd = os.open(path, os.O_RDONLY)  # not open for writing: every pwrite fails
    try:
        with pytest.raises(gms.GmsError) as ei:
            gms.gms_capture_fd(d.m, pipe, fd, 0, None, None)
        assert ei.value.status == gms.ERR_IO
        with pytest.raises(gms.GmsError) as ei:
            gms.gms_capture_fd(d.m, pipe, -1, 0, None, None)
        assert ei.value.status == gms.ERR_ARG
    finally:
        os.close(fd)
    # the pipe and the manifest remain usable after the error; mapped writes were asked for but this descriptor cannot be
    # mapped for writing (write-only), so pwrite is used
    gms.gms_pipe_mapped_writes(pipe, True)
    fd = os.open(path, os.O_WRONLY)
    try:
        st = gms.gms_capture_fd(d.m, pipe, fd, 0, None, None)
        assert st["mapped_io"] == 0
    finally:
        os.close(fd)
    # nor is a file that ends before the image does ever mapped (or extended by the mapping): pwrite grows it
    short = str(tmp_path / "short.bin")
    with open(short, "wb") as f:
        f.write(b"\0" * 4096)
    fd = os.open(short, os.O_RDWR)
    try:
        st = gms.gms_capture_fd(d.m, pipe, fd, 0, None, None)
        assert st["mapped_io"] == 0
    finally:
        os.close(fd)
    for written in (path, short):
        got = np.fromfile(written, dtype=np.uint8)
        for r in w.rows:
            s, o, n = int(r["src_offset"]), int(r["dst_offset"]), int(r["nbytes"])
            assert np.array_equal(got[s:s + n], d.slab[o:o + n].cpu().numpy())
    # tensors that share image bytes cannot be captured
    base = d.slab.data_ptr()
    shared = gms.make_entries([(1, 0, base, 4096), (2, 0, base + 8192, 4096)])
    m2 = gms.gms_manifest_build(shared, 4096)
    fd = os.open(path, os.O_WRONLY)
    try:
        with pytest.raises(gms.GmsError) as ei:
            gms.gms_capture_fd(m2, pipe, fd, 0, None, None)
        assert ei.value.status == gms.ERR_OVERLAP
    finally:
        os.close(fd)
        m2.close()
        pipe.close()
        d.close()


@pytest.mark.gpu
def test_capture_fd_empty_manifest(tmp_path):
    from gpu_harness import payload_of

    w = W.pack_layout("empty", [0, 0], seed=1)
    path = str(tmp_path / "e.bin")
    _write_image(path, np.full(16, PATTERN, np.uint8), 0)
    d = DeviceWorkload(w, image_dev=torch.zeros(16, dtype=torch.uint8, device="cuda"))
    pipe = gms.gms_pipe_create(2, 1 << 20, 1)
    fd = os.open(path, os.O_WRONLY)
    try:
        d.reset_outputs()
        st = gms.gms_capture_fd(d.m, pipe, fd, 0, d.bd_ptr(), d.td_ptr())
        assert st["windows"] == 0 and st["bytes_read"] == 0 and (payload_of(d.td, d.nt) == 0).all()
    finally:
        os.close(fd)
        pipe.close()
        d.close()
    assert (np.fromfile(path, dtype=np.uint8) == PATTERN).all()
