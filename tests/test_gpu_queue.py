"""Dynamic-batch queue on the GPU against its oracle: three detector batches are pushed, pops of
a fixed bz release the oldest items first across batch boundaries, the ring wraps around, and
a small capacity drops the newest items.  Records are compared field by field (bit-exact), the
crops against the oracle's crop of the same rectangle (2e-3)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_01277_b200 as octo
import workloads
from gpu_harness import half_absdiff, make_stage

pytestmark = pytest.mark.gpu

OW, OH = 64, 48


def _run(capacity, bz, pops_between, final_pops, max_wait=-1, options=None):
    wl = workloads.WORKLOADS["traffic_1080p"]
    batches = [workloads.make_batch("traffic_1080p", batch=nb, first_frame=ff) for nb, ff in ((2, 0), (3, 10), (1, 20))]
    st = make_stage(wl, 4, branches=((OW, OH),))
    q = octo.Queue(capacity, OW, OH, max_bz=bz)
    oq = oracle.OracleQueue(capacity)
    if options:
        q.set_options(**options)
    got, want = [], []
    try:
        keep = []

        def pop():
            buf = torch.full((bz, 3, OH, OW), 0x7BFF, dtype=torch.int16, device="cuda")
            _, items, info = q.pop(bz, out=buf.view(torch.float16), max_wait=max_wait)
            torch.cuda.synchronize()
            recs = items.cpu().numpy().view(octo.QITEM_DTYPE).reshape(-1)
            got.append((buf.cpu().numpy().view(np.uint16), recs, tuple(int(v) for v in info.cpu())))
            want.append(oq.pop(bz, max_wait))

        for b, npop in zip(batches, pops_between):
            frames = [torch.from_numpy(f).cuda() for f in b.frames]
            keep.append(frames)
            st.preprocess(frames, b.sizes)
            st.postprocess(torch.from_numpy(b.head).cuda())
            q.push(st, 0)
            ref = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, ((OW, OH),), max_det=wl.max_det,
                                   do_letterbox=False, do_crops=False)
            payload = [(b.frames[i], b.sizes[i], frames[i].data_ptr(), frames[i].stride(0)) for i in range(b.n)]
            oq.push(ref.items[0], ref.rects[0], payload)
            for _ in range(npop):
                pop()
        for _ in range(final_pops):
            pop()
        for (crops, recs, info), (orecs, oinfo) in zip(got, want):
            assert info == oinfo
            for i, (seq, f, j, rect, (pix, (w, h), ptr, pitch)) in enumerate(orecs):
                r = recs[i]
                assert (int(r["seq"]), int(r["frame"]), int(r["det"])) == (seq, f, j)
                assert (int(r["rx0"]), int(r["ry0"]), int(r["rx1"]), int(r["ry1"])) == rect
                assert (int(r["d_data"]), int(r["width"]), int(r["height"]), int(r["pitch_bytes"])) == (ptr, w, h, pitch)
                box = np.zeros(1, dtype=oracle.DET_DTYPE)
                box["x1"], box["y1"], box["x2"], box["y2"] = rect  # integer box -> the same rectangle
                assert oracle.crop_rect(box, w, h) == rect
                assert half_absdiff(crops[i], oracle.crop(pix, w, h, box, OW, OH, **(options or {}))) <= 2e-3
            assert np.all(crops[len(orecs):] == 0x7BFF)
        return want
    finally:
        q.close()
        st.close()


def test_queue_fifo_across_batches_with_wraparound():
    want = _run(capacity=96, bz=32, pops_between=(1, 2, 0), final_pops=4)
    infos = [w[1] for w in want]
    assert infos[0][0] == 32 and infos[-1] == (0, 0, 0, -1)      # full first batch, empty at the end
    assert any(len({r[0] for r in w[0]}) > 1 for w in want)       # some pop spans two pushes
    assert sum(i[0] for i in infos) > 96                          # more items than the ring holds: it wrapped


def test_queue_drops_newest_when_full():
    want = _run(capacity=40, bz=16, pops_between=(0, 0, 0), final_pops=4)
    infos = [w[1] for w in want]
    assert infos[0][2] > 0 and sum(i[0] for i in infos) == 40


def test_queue_release_rule_decided_on_the_device():
    """bz larger than one batch's items: pops right after a push release nothing until the head of
    the queue has waited two pushes or a full batch is pending."""
    want = _run(capacity=256, bz=64, pops_between=(1, 1, 1), final_pops=2, max_wait=2)
    infos = [w[1] for w in want]
    assert infos[0][0] == 0 and infos[0][1] > 0          # first batch alone: not full, not due
    assert any(i[0] == 64 for i in infos) or infos[2][0] > 0
    assert sum(i[0] for i in infos) > 0


def test_queue_with_crop_options():
    _run(capacity=96, bz=32, pops_between=(1, 1, 0), final_pops=2,
         options=dict(keep_aspect=True, mean=(0.485, 0.456, 0.406), std=(0.229, 0.224, 0.225), pad_value=30))
    q = octo.Queue(16, 64, 48, max_bz=8)
    try:
        with pytest.raises(octo.OctoError):
            q.set_options(std=(0.2, 0.0, 0.2))
        with pytest.raises(octo.OctoError):
            q.set_options(pad_value=300)
    finally:
        q.close()


def test_queue_argument_errors():
    from paper_2502_01277_b200 import binding as B
    lib = octo.load_library()
    import ctypes
    h = ctypes.c_void_p()
    for args in ((0, 0, 64, 48, 1, 1), (0, 16, 60, 48, 1, 8), (0, 16, 64, 0, 1, 8), (0, 16, 64, 48, 1, 32),
                 (0, 16, 64, 48, 2, 8)):
        assert lib.octo_queue_create(*args, ctypes.byref(h)) == B.OCTO_E_INVALID_ARG
    q = octo.Queue(16, 64, 48, max_bz=8)
    st = octo.Stage(net_size=64, max_batch=2, num_anchors=252, num_classes=4, max_det=10, branches=((16, 16),))
    try:
        assert lib.octo_queue_push(q.handle, st.handle, 0, None) == B.OCTO_E_NO_PREPROCESS
        out = torch.zeros((8, 3, 48, 64), dtype=torch.float16, device="cuda")
        info = torch.zeros((4,), dtype=torch.int32, device="cuda")
        assert lib.octo_queue_pop(q.handle, 9, out.data_ptr(), None, info.data_ptr(), None) == B.OCTO_E_INVALID_ARG
        assert lib.octo_queue_pop(q.handle, 4, out.data_ptr() + 2, None, info.data_ptr(), None) == B.OCTO_E_ALIGNMENT
        assert lib.octo_queue_pop(q.handle, 4, out.data_ptr(), None, info.data_ptr(), None) == B.OCTO_OK
        torch.cuda.synchronize()
        assert info.tolist() == [0, 0, 0, -1]
    finally:
        q.close()
        st.close()
