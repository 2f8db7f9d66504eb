"""Error paths of the C ABI that need a live stage (so a GPU), all produced on the host:
bad pointers, sizes, alignment and call order.  None of them launches a kernel."""
import numpy as np
import pytest
import torch

import paper_2502_01277_b200 as octo
from paper_2502_01277_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.fixture()
def stage():
    st = octo.Stage(net_size=64, max_batch=2, num_anchors=252, num_classes=4, max_det=10, branches=((16, 16),))
    yield st
    st.close()


def _frame(w=40, h=30, pitch=None):
    pitch = pitch or (3 * w + 15) // 16 * 16
    return torch.zeros((h, pitch), dtype=torch.uint8, device="cuda")


def _code(fn, *a):
    with pytest.raises(octo.OctoError) as ei:
        fn(*a)
    return ei.value.code


def test_preprocess_argument_errors(stage):
    out = torch.empty((2, 3, 64, 64), dtype=torch.float16, device="cuda")
    f = _frame()
    ok = (f.data_ptr(), 40, 30, f.stride(0))
    h = stage.handle
    assert _code(octo.octo_preprocess_batch, h, [], out.data_ptr()) == B.OCTO_E_INVALID_ARG
    assert _code(octo.octo_preprocess_batch, h, [ok] * 3, out.data_ptr()) == B.OCTO_E_CAPACITY
    assert _code(octo.octo_preprocess_batch, h, [ok], 0) == B.OCTO_E_INVALID_ARG
    assert _code(octo.octo_preprocess_batch, h, [ok], out.data_ptr() + 2) == B.OCTO_E_ALIGNMENT
    assert _code(octo.octo_preprocess_batch, h, [(0, 40, 30, 128)], out.data_ptr()) == B.OCTO_E_INVALID_ARG
    assert _code(octo.octo_preprocess_batch, h, [(f.data_ptr(), 0, 30, 128)], out.data_ptr()) == B.OCTO_E_INVALID_ARG
    assert _code(octo.octo_preprocess_batch, h, [(f.data_ptr(), 40, 30, 112)], out.data_ptr()) == B.OCTO_E_INVALID_ARG
    assert _code(octo.octo_preprocess_batch, h, [(f.data_ptr(), 40, 30, 136)], out.data_ptr()) == B.OCTO_E_ALIGNMENT
    assert _code(octo.octo_preprocess_batch, h, [(f.data_ptr() + 8, 40, 30, 128)], out.data_ptr()) == B.OCTO_E_ALIGNMENT
    assert _code(octo.octo_preprocess_batch, h, [(f.data_ptr(), 20000, 30, 60000)], out.data_ptr()) == B.OCTO_E_CAPACITY
    assert stage.launch_count == 0


def test_call_order_errors(stage):
    head = torch.zeros((1, 252, 9), dtype=torch.float32, device="cuda")
    dets = torch.zeros((1, 10, 32), dtype=torch.uint8, device="cuda")
    counts = torch.zeros((1,), dtype=torch.int32, device="cuda")
    crops = torch.zeros((4, 3, 16, 16), dtype=torch.float16, device="cuda")
    off = torch.zeros((3,), dtype=torch.int32, device="cuda")
    ni = torch.zeros((2,), dtype=torch.int32, device="cuda")
    h = stage.handle
    assert _code(octo.octo_postprocess_batch, h, head.data_ptr(), 1, dets.data_ptr(), counts.data_ptr()) == B.OCTO_E_NO_PREPROCESS
    assert _code(octo.octo_crop_batch, h, 0, 0, 4, crops.data_ptr(), off.data_ptr(), ni.data_ptr()) == B.OCTO_E_NO_PREPROCESS
    f = _frame()
    stage.preprocess([f], [(40, 30)])
    assert _code(octo.octo_crop_batch, h, 0, 0, 4, crops.data_ptr(), off.data_ptr(), ni.data_ptr()) == B.OCTO_E_NO_POSTPROCESS
    assert _code(octo.octo_postprocess_batch, h, head.data_ptr(), 2, dets.data_ptr(), counts.data_ptr()) == B.OCTO_E_INVALID_ARG
    assert _code(octo.octo_postprocess_batch, h, 0, 1, dets.data_ptr(), counts.data_ptr()) == B.OCTO_E_INVALID_ARG
    stage.postprocess(head, dets=dets, counts=counts)
    assert _code(octo.octo_crop_batch, h, 1, 0, 4, crops.data_ptr(), off.data_ptr(), ni.data_ptr()) == B.OCTO_E_INVALID_ARG
    assert _code(octo.octo_crop_batch, h, 0, -1, 4, crops.data_ptr(), off.data_ptr(), ni.data_ptr()) == B.OCTO_E_INVALID_ARG
    assert _code(octo.octo_crop_batch, h, 0, 0, 4, crops.data_ptr() + 2, off.data_ptr(), ni.data_ptr()) == B.OCTO_E_ALIGNMENT
    assert _code(octo.octo_crop_batch, h, 0, 0, 4, 0, off.data_ptr(), ni.data_ptr()) == B.OCTO_E_INVALID_ARG
    # a zero-slot window is legal: offsets and totals only
    octo.octo_crop_batch(h, 0, 0, 0, 0, off.data_ptr(), ni.data_ptr())
    torch.cuda.synchronize()
    assert ni.tolist() == [0, 0] and off.tolist()[:2] == [0, 0]
    # a new preprocess invalidates the detections of the previous batch
    stage.preprocess([f], [(40, 30)])
    assert _code(octo.octo_crop_batch, h, 0, 0, 4, crops.data_ptr(), off.data_ptr(), ni.data_ptr()) == B.OCTO_E_NO_POSTPROCESS


def test_workspace_and_stats(stage):
    assert stage.workspace_bytes > 0
    s = stage.stats()
    assert s["candidates"] == 0 and s["kept"] == 0 and s["status_word"] == 0
    assert stage.status() == 0


def test_repeated_passes_are_bit_identical():
    """Candidate append order, tile hand-out and the scheduler words change from launch to launch;
    the results must not: 40 passes over the same batch, two stages interleaved on two streams."""
    import numpy as np
    import workloads
    from gpu_harness import make_stage

    b = workloads.make_batch("traffic_1080p", batch=3)
    wl = b.workload
    dev = torch.device("cuda", 0)
    stages = [make_stage(wl, b.n), make_stage(wl, b.n)]
    streams = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    try:
        frames = [torch.from_numpy(f).to(dev) for f in b.frames]
        head = torch.from_numpy(b.head).to(dev)
        first = None
        for it in range(40):
            st, s = stages[it % 2], streams[it % 2]
            with torch.cuda.stream(s):
                det_in = st.preprocess(frames, b.sizes, stream=s)
                dets, counts = st.postprocess(head, stream=s)
                crops, offsets, n_items = st.crop(0, 200, stream=s)
                crops2, _, _ = st.crop(0, 7, first_item=5, stream=s)  # a second window on the same stage
            s.synchronize()
            packed = int(n_items[0])
            c = counts.cpu().numpy()
            d = dets.cpu().numpy()
            kept = np.concatenate([d[i, :c[i]] for i in range(b.n)])  # records beyond the counts are not written
            cur = (det_in.view(torch.int16).cpu().numpy(), kept, c,
                   crops[:packed].view(torch.int16).cpu().numpy(), offsets.cpu().numpy(),
                   crops2.view(torch.int16).cpu().numpy())
            if first is None:
                first = cur
                assert packed > 20
            else:
                for x, y in zip(cur, first):
                    assert np.array_equal(x, y)
            assert np.array_equal(cur[5], cur[3][5:12])
            assert st.status(s) & ~0x2 == 0  # the small second window is truncated by design
    finally:
        for st in stages:
            st.close()


def test_two_host_threads_drive_two_stages():
    """Stage objects share no host state: two threads, each with a stage, a stream and a batch of
    its own (different frame sizes, so a mixed-up frame table would move every box), run 200 passes
    side by side on one GPU; every pass of both must give the oracle's detections, the last one
    also its rectangles and crops."""
    import threading
    from dataclasses import replace

    import oracle
    import workloads
    from gpu_harness import half_absdiff

    passes = 200
    dev = torch.device("cuda", 0)
    specs = [(replace(workloads.WORKLOADS["traffic_1080p"], frame_sizes=((640, 360),), branches=((64, 64),)), 2, 71),
             (replace(workloads.WORKLOADS["traffic_1080p"], frame_sizes=((1280, 720),), branches=((96, 32),)), 3, 72)]
    jobs, errors = [], []
    for wl, n, seed in specs:
        b = workloads.make_batch(wl, batch=n, seed=seed)
        ref = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, max_det=wl.max_det,
                               do_letterbox=False, threads=4)
        st = octo.Stage(net_size=wl.net_size, max_batch=n, num_anchors=wl.num_anchors, num_classes=wl.num_classes,
                        max_det=wl.max_det, branches=wl.branches)
        stream = torch.cuda.Stream(dev)
        with torch.cuda.stream(stream):
            frames = [torch.from_numpy(f).to(dev) for f in b.frames]
            head = torch.from_numpy(b.head).to(dev)
            det_in = torch.empty((n, 3, wl.net_size, wl.net_size), dtype=torch.float16, device=dev)
            dets = torch.zeros((passes, n, wl.max_det, 32), dtype=torch.uint8, device=dev)
            counts = torch.full((passes, n), -1, dtype=torch.int32, device=dev)
            cap = len(ref.items[0]) + 2
            ow, oh = wl.branches[0]
            crops = torch.zeros((cap, 3, oh, ow), dtype=torch.float16, device=dev)
            offs = torch.zeros((n + 1,), dtype=torch.int32, device=dev)
            ni = torch.zeros((2,), dtype=torch.int32, device=dev)
        stream.synchronize()
        jobs.append(dict(b=b, ref=ref, st=st, stream=stream, frames=frames, head=head, det_in=det_in, dets=dets,
                         counts=counts, crops=crops, offs=offs, ni=ni, cap=cap))
    start = threading.Barrier(len(jobs))

    def work(j):
        try:
            torch.cuda.set_device(dev)
            start.wait()
            for k in range(passes):
                j["st"].preprocess(j["frames"], j["b"].sizes, out=j["det_in"], stream=j["stream"])
                j["st"].postprocess(j["head"], dets=j["dets"][k], counts=j["counts"][k], stream=j["stream"])
                j["st"].crop(0, j["cap"], out=j["crops"], offsets=j["offs"], n_items=j["ni"], stream=j["stream"])
            j["stream"].synchronize()
        except Exception as e:  # pragma: no cover
            errors.append(e)

    threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
    try:
        for t in threads:
            t.start()
        for t in threads:
            t.join()
        assert not errors, errors
        for j in jobs:
            ref, n = j["ref"], j["b"].n
            counts = j["counts"].cpu().numpy()
            dets = j["dets"].cpu().numpy().view(octo.DET_DTYPE).reshape(passes, n, -1)
            assert np.all(counts == ref.counts[None, :])
            for i, k in enumerate(ref.counts):
                want = ref.dets[i, :k].tobytes()
                for p in range(passes):
                    assert dets[p, i, :k].tobytes() == want, f"pass {p}, frame {i}"
            packed, total = (int(v) for v in j["ni"].cpu())
            assert packed == total == len(ref.items[0])
            it = j["st"].item_table(0, packed)
            assert np.array_equal(np.stack([it["rx0"], it["ry0"], it["rx1"], it["ry1"]], 1), ref.rects[0])
            got = j["crops"][:packed].view(torch.int16).cpu().numpy().view(np.uint16)
            assert half_absdiff(got, ref.crops[0]) <= 2e-3
            assert j["st"].status(j["stream"]) == 0
    finally:
        for j in jobs:
            j["st"].close()


def test_a_wait_that_runs_out_is_reported_and_cleared(stage):
    """The time-out path of the bounded device waits, made to run out without any copy in flight:
    the self-test kernel arms a barrier for bytes nobody sends and gives up after a few hundred
    polls.  The status word carries the bit, octo_stage_status reports OCTO_E_DEVICE_TIMEOUT, the
    context stays usable, and clearing the word brings the stage back to OCTO_OK."""
    lib = octo.load_library()
    import ctypes
    w = ctypes.c_uint32(0)
    assert lib.octo_stage_status(stage.handle, ctypes.byref(w), None) == B.OCTO_OK and w.value == 0
    stage.selftest_wait(polls=300)
    rc = lib.octo_stage_status(stage.handle, ctypes.byref(w), None)
    assert rc == B.OCTO_E_DEVICE_TIMEOUT and w.value & B.OCTO_STATUS_COPY_TIMEOUT
    assert octo.octo_stage_status(stage.handle) & B.OCTO_STATUS_COPY_TIMEOUT
    stage.clear_status()
    assert lib.octo_stage_status(stage.handle, ctypes.byref(w), None) == B.OCTO_OK and w.value == 0
    # the stage still works
    f = _frame()
    out = stage.preprocess([f], [(40, 30)])
    torch.cuda.synchronize()
    assert stage.status() == 0 and out.shape == (1, 3, 64, 64)
    assert lib.octo_stage_selftest_wait(stage.handle, 0, None) == B.OCTO_E_INVALID_ARG
    assert lib.octo_stage_selftest_wait(None, 10, None) == B.OCTO_E_INVALID_ARG


def test_kernel_timing_counts_every_launch_and_resets(stage):
    """octo_stage_set_timing / octo_stage_kernel_times: with timing on, every kernel launch of the
    batch calls is bracketed by an event pair; the getter sums them per kernel, synchronises, and
    starts from zero again.  With timing off nothing is recorded."""
    f = _frame()
    head = torch.zeros((1, 252, 9), dtype=torch.float32, device="cuda")

    def one_pass():
        stage.preprocess([f], [(40, 30)])
        stage.postprocess(head)
        stage.crop(0, 4)

    one_pass()  # untimed
    t = stage.kernel_times()
    assert all(t[k] == (0.0, 0) for k in B.KERNEL_NAMES) and t["dropped"] == 0
    stage.set_timing(True)
    before = stage.launch_count
    for _ in range(3):
        one_pass()
    t = stage.kernel_times()
    launched = {k: v[1] for k, v in t.items() if k != "dropped" and v[1]}
    assert launched == {"letterbox": 3, "decode": 3, "nms": 3, "crop": 3}
    assert sum(launched.values()) == stage.launch_count - before
    assert all(0.0 < t[k][0] < 50.0 for k in launched) and t["dropped"] == 0
    t = stage.kernel_times()  # the getter reset the record
    assert all(t[k] == (0.0, 0) for k in B.KERNEL_NAMES)
    stage.set_timing(False)
    one_pass()
    t = stage.kernel_times()
    assert all(t[k] == (0.0, 0) for k in B.KERNEL_NAMES)
