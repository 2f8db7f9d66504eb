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
