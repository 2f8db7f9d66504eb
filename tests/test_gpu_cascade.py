"""Second-level cascade on the GPU against the oracle: a first-level detector stage crops its
survivors to 256x256 (the plate-detector branch of the traffic pipeline); a chained stage
adopts those crops as its detector input, decodes its own synthetic head, maps the boxes back
into the ORIGINAL frame through the upstream rectangles and crops again from the original
pixels.  Indices, counts, packing, rectangles, scores and box coordinates must be bit-exact;
fp16 pixels within 2e-3."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import paper_2502_01277_b200 as octo
import workloads
from gpu_harness import half_absdiff
from oracle import DET_DTYPE

pytestmark = pytest.mark.gpu


MEAN, STD = (0.485, 0.456, 0.406), (0.229, 0.224, 0.225)


@pytest.mark.parametrize("layout2,opts2", [("rows", None), ("planes", {"keep_aspect": True, "mean": MEAN, "std": STD})])
def test_two_level_cascade_matches_oracle(layout2, opts2):
    """Second level with a row head and plain crops, and with an anchor-free planes head whose
    crops keep their aspect ratio and are normalised."""
    wl = replace(workloads.WORKLOADS["traffic_1080p"], branches=((256, 256),))
    b = workloads.make_batch(wl, batch=3, seed=31)
    s2, c2, max_det2 = 256, 6, 12
    a2 = workloads.num_anchors(s2)
    # ---- level 1 on the GPU
    st1 = octo.Stage(net_size=wl.net_size, max_batch=b.n, num_anchors=wl.num_anchors, num_classes=wl.num_classes,
                     max_det=wl.max_det, branches=wl.branches)
    st2 = None
    try:
        frames = [torch.from_numpy(f).cuda() for f in b.frames]
        st1.preprocess(frames, b.sizes)
        st1.postprocess(torch.from_numpy(b.head).cuda())
        crops1, off1, ni1 = st1.crop(0, 256)
        torch.cuda.synchronize()
        n1 = int(ni1[0])
        items1 = st1.item_table(0, n1)
        ref1 = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, max_det=wl.max_det,
                                do_letterbox=False)
        assert n1 == len(ref1.items[0]) and n1 > 20
        assert np.array_equal(np.stack([items1["rx0"], items1["ry0"], items1["rx1"], items1["ry1"]], 1),
                              ref1.rects[0])
        # ---- level 2: the 256x256 crops are the detector input; heads are synthetic
        head2 = workloads.make_heads(77, n1, s2, num_classes=c2, n_raised=14, n_groups=4)
        if layout2 == "planes":
            head2 = np.stack([workloads.rows_to_planes(h) for h in head2])
        st2 = octo.Stage(net_size=s2, max_batch=n1, num_anchors=a2, num_classes=c2, max_det=max_det2,
                         branches=((64, 32),), head_layout=layout2, crop_options=[opts2])
        st2.adopt_regions(frames, b.sizes, items1)
        dets2, counts2 = st2.postprocess(torch.from_numpy(head2).cuda())
        cap2 = n1 * max_det2
        buf = torch.full((cap2, 3, 32, 64), 0x7BFF, dtype=torch.int16, device="cuda")
        _, off2, ni2 = st2.crop(0, cap2, out=buf.view(torch.float16))
        torch.cuda.synchronize()
        d2, c2n = octo.dets_to_numpy(dets2, counts2)
        packed2, total2 = (int(v) for v in ni2.cpu())
        items2 = st2.item_table(0, packed2)
        got = buf.cpu().numpy().view(np.uint16)
        assert st2.status() == 0
        # ---- oracle chain
        ref_d = np.zeros((n1, max_det2), dtype=DET_DTYPE)
        ref_c = np.zeros(n1, dtype=np.int32)
        for i in range(n1):
            r = ref1.rects[0][i]
            d, _ = oracle.postprocess_region(head2[i], tuple(int(v) for v in r), s2, max_det=max_det2, layout=layout2)
            ref_d[i, : len(d)] = d
            ref_c[i] = len(d)
        assert np.array_equal(c2n, ref_c) and int(ref_c.sum()) > n1
        for i in range(n1):
            k = ref_c[i]
            assert d2[i, :k].tobytes() == ref_d[i, :k].tobytes(), f"item {i}: detections differ"
            rx0, ry0, rx1, ry1 = ref1.rects[0][i]
            assert np.all((ref_d[i, :k]["x1"] >= rx0) & (ref_d[i, :k]["x2"] <= rx1))
            assert np.all((ref_d[i, :k]["y1"] >= ry0) & (ref_d[i, :k]["y2"] <= ry1))
        offs, its, (pk, tot) = oracle.assemble(ref_d, ref_c, max_det2)
        assert (packed2, total2) == (pk, tot) and np.array_equal(off2.cpu().numpy(), offs)
        assert np.array_equal(np.stack([items2["frame"], items2["det"]], 1), its)
        for k, (i, j) in enumerate(its):
            f = int(items1["frame"][i])  # the ORIGINAL frame behind upstream item i
            w, h = b.sizes[f]
            rect = oracle.crop_rect(ref_d[i, j], w, h)
            assert (int(items2["rx0"][k]), int(items2["ry0"][k]), int(items2["rx1"][k]), int(items2["ry1"][k])) == rect
            want = oracle.crop(b.frames[f], w, h, ref_d[i, j], 64, 32, **(opts2 or {}))
            assert half_absdiff(got[k], want) <= 2e-3
        assert np.all(got[packed2:] == 0x7BFF)
    finally:
        st1.close()
        if st2 is not None:
            st2.close()


def test_device_hand_off_equals_the_host_hand_off_and_the_oracle():
    """octo_adopt_items_device: the chained stage reads the upstream item table on the device, with
    no synchronisation in between.  The level-2 batch is provisioned larger than the number of
    upstream items: the surplus entries (fed with a head full of raised candidates) must yield no
    detections.  A window that starts inside the item table is taken as well."""
    wl = replace(workloads.WORKLOADS["traffic_1080p"], branches=((256, 256),))
    b = workloads.make_batch(wl, batch=3, seed=33)
    s2, c2, max_det2 = 256, 6, 12
    a2 = workloads.num_anchors(s2)
    ref1 = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, max_det=wl.max_det,
                            do_letterbox=False, do_crops=False)
    n1 = len(ref1.items[0])
    assert n1 > 20
    bz = n1 + 5                      # downstream batch size: five surplus entries
    head2 = workloads.make_heads(78, bz, s2, num_classes=c2, n_raised=14, n_groups=4)
    st1 = octo.Stage(net_size=wl.net_size, max_batch=b.n, num_anchors=wl.num_anchors, num_classes=wl.num_classes,
                     max_det=wl.max_det, branches=wl.branches)
    st2 = octo.Stage(net_size=s2, max_batch=bz, num_anchors=a2, num_classes=c2, max_det=max_det2, branches=((64, 32),))
    stream = torch.cuda.Stream()
    try:
        with torch.cuda.stream(stream):
            frames = [torch.from_numpy(f).cuda() for f in b.frames]
            d_head1, d_head2 = torch.from_numpy(b.head).cuda(), torch.from_numpy(head2).cuda()
        stream.synchronize()
        for first in (0, 7):
            m = bz - first           # entries of this level-2 batch (n1 - first of them are real)
            cap2 = m * max_det2
            # both levels are enqueued back to back: nothing reads the device in between
            st1.preprocess(frames, b.sizes, stream=stream)
            st1.postprocess(d_head1, stream=stream)
            crops1, off1, ni1 = st1.crop(0, 256, stream=stream)
            st2.adopt_items_device(st1, 0, m, first=first, stream=stream)
            dets2, counts2 = st2.postprocess(d_head2[first:], stream=stream)
            with torch.cuda.stream(stream):
                buf = torch.full((cap2, 3, 32, 64), 0x7BFF, dtype=torch.int16, device="cuda")
            _, off2, ni2 = st2.crop(0, cap2, out=buf.view(torch.float16), stream=stream)
            stream.synchronize()
            assert int(ni1[0]) == n1
            d2, c2n = octo.dets_to_numpy(dets2, counts2)
            packed2, total2 = (int(v) for v in ni2.cpu())
            items2 = st2.item_table(0, packed2)
            got = buf.cpu().numpy().view(np.uint16)
            assert st2.status(stream) == 0 and st1.status(stream) == 0
            ref_d = np.zeros((m, max_det2), dtype=DET_DTYPE)
            ref_c = np.zeros(m, dtype=np.int32)
            for i in range(n1 - first):
                r = ref1.rects[0][first + i]
                d, _ = oracle.postprocess_region(head2[first + i], tuple(int(v) for v in r), s2, max_det=max_det2)
                ref_d[i, : len(d)] = d
                ref_c[i] = len(d)
            assert np.array_equal(c2n, ref_c) and np.all(c2n[n1 - first:] == 0) and int(ref_c.sum()) > n1 - first
            for i in range(m):
                assert d2[i, : ref_c[i]].tobytes() == ref_d[i, : ref_c[i]].tobytes(), f"entry {i}: detections differ"
            offs, its, (pk, tot) = oracle.assemble(ref_d, ref_c, max_det2)
            assert (packed2, total2) == (pk, tot) and np.array_equal(off2.cpu().numpy(), offs)
            assert np.array_equal(np.stack([items2["frame"], items2["det"]], 1), its)
            for k, (i, j) in enumerate(its):
                f = int(ref1.items[0][first + i][0])  # the ORIGINAL frame behind upstream item first + i
                w, h = b.sizes[f]
                rect = oracle.crop_rect(ref_d[i, j], w, h)
                assert (int(items2["rx0"][k]), int(items2["ry0"][k]), int(items2["rx1"][k]),
                        int(items2["ry1"][k])) == rect
                assert half_absdiff(got[k], oracle.crop(b.frames[f], w, h, ref_d[i, j], 64, 32)) <= 2e-3
            assert np.all(got[packed2:] == 0x7BFF)
    finally:
        st1.close()
        st2.close()


def test_three_levels_chained_on_the_device():
    """frames -> detector -> 128x128 crops -> chained detector -> 64x64 crops -> chained detector:
    the third stage adopts items of a stage whose own frame table already lives on the device.
    Boxes of every level are in ORIGINAL-frame pixels and clamped to the rectangle above them."""
    wl = replace(workloads.WORKLOADS["traffic_1080p"], frame_sizes=((1280, 720),), branches=((128, 128),),
                 n_raised=40, n_groups=6)
    b = workloads.make_batch(wl, batch=2, seed=35)
    s2, s3, c, md2, md3 = 128, 64, 5, 6, 4
    a2, a3 = workloads.num_anchors(s2), workloads.num_anchors(s3)
    ref1 = oracle.run_stage(b.frames, b.sizes, b.head, wl.net_size, wl.branches, max_det=wl.max_det,
                            do_letterbox=False, do_crops=False)
    n1 = len(ref1.items[0])
    assert n1 > 8
    head2 = workloads.make_heads(80, n1, s2, num_classes=c, n_raised=10, n_groups=3)
    # level 2 in the oracle: detections per upstream item, then its item list
    d2 = np.zeros((n1, md2), dtype=DET_DTYPE)
    c2 = np.zeros(n1, dtype=np.int32)
    for i in range(n1):
        d, _ = oracle.postprocess_region(head2[i], tuple(int(v) for v in ref1.rects[0][i]), s2, max_det=md2)
        d2[i, : len(d)] = d
        c2[i] = len(d)
    _, its2, (n2, _) = oracle.assemble(d2, c2, md2)
    assert n2 > n1
    rects2 = [oracle.crop_rect(d2[i, j], *b.sizes[int(ref1.items[0][i][0])]) for i, j in its2]
    head3 = workloads.make_heads(81, n2, s3, num_classes=c, n_raised=8, n_groups=2)
    st1 = octo.Stage(net_size=wl.net_size, max_batch=b.n, num_anchors=wl.num_anchors, num_classes=wl.num_classes,
                     max_det=wl.max_det, branches=wl.branches)
    st2 = octo.Stage(net_size=s2, max_batch=n1, num_anchors=a2, num_classes=c, max_det=md2, branches=((s3, s3),))
    st3 = octo.Stage(net_size=s3, max_batch=n2, num_anchors=a3, num_classes=c, max_det=md3, branches=((32, 32),))
    try:
        frames = [torch.from_numpy(f).cuda() for f in b.frames]
        st1.preprocess(frames, b.sizes)
        st1.postprocess(torch.from_numpy(b.head).cuda())
        st1.crop(0, n1 + 4)
        st2.adopt_items_device(st1, 0, n1)
        st2.postprocess(torch.from_numpy(head2).cuda())
        _, _, ni2 = st2.crop(0, n1 * md2)
        st3.adopt_items_device(st2, 0, n2)
        dets3, counts3 = st3.postprocess(torch.from_numpy(head3).cuda())
        buf = torch.full((n2 * md3, 3, 32, 32), 0x7BFF, dtype=torch.int16, device="cuda")
        _, off3, ni3 = st3.crop(0, n2 * md3, out=buf.view(torch.float16))
        torch.cuda.synchronize()
        assert int(ni2[0]) == n2
        d3, c3 = octo.dets_to_numpy(dets3, counts3)
        ref_d = np.zeros((n2, md3), dtype=DET_DTYPE)
        ref_c = np.zeros(n2, dtype=np.int32)
        for k in range(n2):
            d, _ = oracle.postprocess_region(head3[k], rects2[k], s3, max_det=md3)
            ref_d[k, : len(d)] = d
            ref_c[k] = len(d)
            rx0, ry0, rx1, ry1 = rects2[k]
            assert np.all((d["x1"] >= rx0) & (d["x2"] <= rx1) & (d["y1"] >= ry0) & (d["y2"] <= ry1))
        assert np.array_equal(c3, ref_c) and int(ref_c.sum()) > 0
        for k in range(n2):
            assert d3[k, : ref_c[k]].tobytes() == ref_d[k, : ref_c[k]].tobytes(), f"level-2 item {k}"
        offs, its3, (pk, tot) = oracle.assemble(ref_d, ref_c, md3)
        assert tuple(int(v) for v in ni3.cpu()) == (pk, tot) and np.array_equal(off3.cpu().numpy(), offs)
        items3 = st3.item_table(0, pk)
        got = buf.cpu().numpy().view(np.uint16)
        for q, (k, j) in enumerate(its3):
            f = int(ref1.items[0][its2[k][0]][0])  # the original frame two levels up
            w, h = b.sizes[f]
            assert (int(items3["rx0"][q]), int(items3["ry0"][q]), int(items3["rx1"][q]),
                    int(items3["ry1"][q])) == oracle.crop_rect(ref_d[k, j], w, h)
            assert half_absdiff(got[q], oracle.crop(b.frames[f], w, h, ref_d[k, j], 32, 32)) <= 2e-3
        for st in (st1, st2, st3):
            assert st.status() == 0
    finally:
        st1.close()
        st2.close()
        st3.close()


def test_adopt_items_device_argument_errors():
    from paper_2502_01277_b200 import binding as B
    lib = octo.load_library()
    up = octo.Stage(net_size=64, max_batch=2, num_anchors=252, num_classes=4, max_det=10, branches=((32, 32), (16, 16)))
    st = octo.Stage(net_size=32, max_batch=4, num_anchors=63, num_classes=4, max_det=5, branches=((8, 8),))
    try:
        call = lambda s, u, br, first, n: lib.octo_adopt_items_device(s, u, br, first, n, None)  # noqa: E731
        assert call(st.handle, up.handle, 0, 0, 2) == B.OCTO_E_NO_PREPROCESS      # upstream has no batch yet
        f = torch.zeros((30, 128), dtype=torch.uint8, device="cuda")
        up.preprocess([f], [(40, 30)])
        assert call(st.handle, up.handle, 0, 0, 2) == B.OCTO_E_NO_POSTPROCESS     # branch 0 never cropped
        up.postprocess(torch.full((1, 252, 9), -9.0, device="cuda"))
        up.crop(0, 4)
        up.crop(1, 4)
        assert call(st.handle, up.handle, 0, 0, 4) == B.OCTO_OK
        assert call(st.handle, up.handle, 0, 0, 5) == B.OCTO_E_CAPACITY           # n > max_batch
        assert call(st.handle, up.handle, 0, 19, 4) == B.OCTO_E_CAPACITY          # window past the item table
        assert call(st.handle, up.handle, 1, 0, 2) == B.OCTO_E_INVALID_ARG        # branch is not net_size wide
        assert call(st.handle, up.handle, 2, 0, 2) == B.OCTO_E_INVALID_ARG
        assert call(st.handle, up.handle, 0, -1, 2) == B.OCTO_E_INVALID_ARG
        assert call(st.handle, up.handle, 0, 0, 0) == B.OCTO_E_INVALID_ARG
        assert call(st.handle, st.handle, 0, 0, 2) == B.OCTO_E_INVALID_ARG
        assert call(None, up.handle, 0, 0, 2) == B.OCTO_E_INVALID_ARG
        torch.cuda.synchronize()
    finally:
        st.close()
        up.close()


def test_adopt_regions_argument_errors():
    from paper_2502_01277_b200 import binding as B
    st = octo.Stage(net_size=64, max_batch=2, num_anchors=252, num_classes=4, max_det=10, branches=((16, 16),))
    try:
        f = torch.zeros((30, 128), dtype=torch.uint8, device="cuda")
        lib = octo.load_library()

        def call(rects, n=None):
            arr = (B.Region * max(len(rects), 1))()
            for i, (ptr, w, h, p, r) in enumerate(rects):
                arr[i].d_data, arr[i].width, arr[i].height, arr[i].pitch_bytes = ptr, w, h, p
                arr[i].rx0, arr[i].ry0, arr[i].rx1, arr[i].ry1 = r
            return lib.octo_adopt_regions(st.handle, arr, len(rects) if n is None else n, None)

        ok = (f.data_ptr(), 40, 30, 128, (2, 3, 20, 25))
        assert call([ok]) == B.OCTO_OK
        assert call([ok], n=0) == B.OCTO_E_INVALID_ARG
        assert call([ok] * 3) == B.OCTO_E_CAPACITY
        assert call([(f.data_ptr(), 40, 30, 128, (5, 3, 5, 25))]) == B.OCTO_E_INVALID_ARG   # empty
        assert call([(f.data_ptr(), 40, 30, 128, (5, 3, 41, 25))]) == B.OCTO_E_INVALID_ARG  # outside the frame
        assert call([(f.data_ptr(), 40, 30, 112, (2, 3, 20, 25))]) == B.OCTO_E_INVALID_ARG  # pitch < 3 w
        assert call([(f.data_ptr() + 4, 40, 30, 128, (2, 3, 20, 25))]) == B.OCTO_E_ALIGNMENT
        assert call([(0, 40, 30, 128, (2, 3, 20, 25))]) == B.OCTO_E_INVALID_ARG
    finally:
        st.close()
