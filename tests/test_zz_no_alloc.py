"""st_agreement_noalloc: the agreement measurement for callers that cannot allocate device memory
(a process whose memory pool owns all of HBM, a loop that cannot take cudaMalloc's device-wide
synchronisation, code running while allocation calls are forbidden).  It must give exactly the counts
and the mean IoU of the ordinary st_agreement, also on a second call in a row, because both calls
share one fixed array inside the library that has to be cleared each time.

Collected last on purpose (file name): a run that stops at the first failure has then already run
every other test."""
import numpy as np
import pytest

import paper_2003_10735_b200 as st

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _masks(seed, C, h, w):
    rng = np.random.default_rng(seed)
    P = 16 * h * w
    lab = np.repeat(rng.integers(0, C, P // 8 + 1), 8)[:P].astype(np.uint8)
    pred = np.where(rng.random(P) < 0.6, lab, rng.integers(0, C, P)).astype(np.uint8)
    return lab.reshape(4 * h, 4 * w), pred.reshape(4 * h, 4 * w)


def test_noalloc_matches_st_agreement_on_two_calls_in_a_row():
    C, h, w = 21, 45, 80
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        ctx = st.st_init_head(n_streams=1, c_in=8, c_hidden=0, n_classes=C, feat_h=h, feat_w=w,
                              cuda_stream=stream.cuda_stream,
                              init_params=np.zeros(st.st_param_count(8, 0, C), np.float32))
        conf_new = torch.empty((C, C), dtype=torch.int64, device="cuda")
        miou_new = torch.empty(1, dtype=torch.float64, device="cuda")
        for call, seed in enumerate((1, 2)):              # different masks: stale counts would show
            lab, pred = _masks(seed, C, h, w)
            d_lab, d_pred = torch.from_numpy(lab).cuda(), torch.from_numpy(pred).cuda()
            conf_ref = torch.zeros((C, C), dtype=torch.int64, device="cuda")
            miou_ref = st.st_agreement(ctx, 0, d_pred, d_lab, conf_ref)
            st.st_agreement_noalloc(d_pred, d_lab, C, stream.cuda_stream, conf_new, miou_new)
            stream.synchronize()
            assert torch.equal(conf_new, conf_ref), f"call {call}"            # integer counts: bit-exact
            assert miou_new.item() == miou_ref, f"call {call}"                 # same counts, same arithmetic
            assert int(conf_new.sum().item()) == lab.size
        st.st_destroy(ctx)


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    d = torch.zeros(64, dtype=torch.uint8, device="cuda")
    conf = torch.zeros((65, 65), dtype=torch.int64, device="cuda")
    miou = torch.zeros(1, dtype=torch.float64, device="cuda")
    with pytest.raises(st.StError) as ei:
        st.st_agreement_noalloc(d, d, st.ST_NOALLOC_MAX_CLASSES + 1, 0, conf, miou)
    assert ei.value.status == st.ST_ERR_UNSUPPORTED
    with pytest.raises(st.StError) as ei:
        st.st_agreement_noalloc(d, d, 1, 0, conf, miou)
    assert ei.value.status == st.ST_ERR_INVALID_ARG


def test_noalloc_allocates_nothing_and_takes_any_length_and_address():
    """Once the first call on the device has looked the internal array up, a call leaves the device's free memory
    as it found it.  Masks whose length is not a multiple of 16 and that start at an odd address go through the
    kernel's pixel-by-pixel path and are checked against a count made with numpy."""
    C, n = 7, 16 * 1000 + 11
    rng = np.random.default_rng(5)
    lab = rng.integers(0, C, n).astype(np.uint8)
    pred = np.where(rng.random(n) < 0.5, lab, rng.integers(0, C, n)).astype(np.uint8)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        raw_l = torch.zeros(n + 16, dtype=torch.uint8, device="cuda")
        raw_p = torch.zeros(n + 16, dtype=torch.uint8, device="cuda")
        d_lab, d_pred = raw_l[1:1 + n], raw_p[3:3 + n]
        d_lab.copy_(torch.from_numpy(lab).cuda()); d_pred.copy_(torch.from_numpy(pred).cuda())
        assert d_lab.data_ptr() % 2 == 1 and d_pred.data_ptr() % 2 == 1
        conf = torch.empty((C, C), dtype=torch.int64, device="cuda")
        miou = torch.empty(1, dtype=torch.float64, device="cuda")
        st.st_agreement_noalloc(d_pred, d_lab, C, stream.cuda_stream, conf, miou)     # the set-up call, if none came before
        stream.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        st.st_agreement_noalloc(d_pred, d_lab, C, stream.cuda_stream, conf, miou)
        stream.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
    ref = np.bincount(lab.astype(np.int64) * C + pred, minlength=C * C).reshape(C, C)
    np.testing.assert_array_equal(conf.cpu().numpy(), ref)
    rows, cols, diag = ref.sum(1), ref.sum(0), np.diag(ref)
    present = rows > 0
    assert miou.item() == pytest.approx(float(np.mean(diag[present] / (rows + cols - diag)[present])), rel=1e-14)
