"""The pieces around a key frame working together on a drifting synthetic clip: the server's loop (Algorithm 3:
teacher labels, Train, pack), the client's key-frame schedule (Algorithm 4 with NextStride of Algorithm 2, the update
arriving before the next frame) and ApplyUpdate, through the C ABI, against the same loop written with the oracle.

The clip: a Voronoi class map translated by a fixed step per frame, teacher logits = noise + 4 on the map's class,
frozen features = ReLU noise + a bump on the channel of the class under each feature pixel (so that the trainable part
can learn the frame and still generalises to the next ones while the scene moves slowly).  The seed is chosen so that
the oracle's decisions (metric against THRESHOLD, the floor in NextStride) keep a margin of more than ten pixels'
worth of mean IoU, which the fp32 path's rounding does not reach.
"""
import numpy as np
import pytest

import oracle
import oracle.schedule as osched
import synth_inputs as si
import paper_2003_10735_b200 as st

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

C_IN, C, FH, FW = 16, 5, 24, 32
N_FRAMES, SEED = 48, 2
THRESHOLD, MAX_UPDATES, MIN_STRIDE, MAX_STRIDE = 0.75, 8, 3, 16
LR, MOMENTUM = 0.1, 0.9


def clip():
    H, W = 4 * FH, 4 * FW
    yy, xx = np.meshgrid(np.arange(H), np.arange(W), indexing="ij")
    frames = []
    for f in range(N_FRAMES):
        cls = si.voronoi_map(H, W, 7, C, 3000 + SEED, shift=(2 * f, f))
        feat = si.label_informed_features(C_IN, FH, FW, cls, 4, 100 * SEED + f, 3.0)
        T = np.random.default_rng(7000 + 100 * SEED + f).normal(0, 1, (C, H, W)).astype(np.float32)
        T[cls, yy, xx] += np.float32(4.0)
        frames.append((feat, T))
    return frames


def oracle_loop(frames, theta):
    head = oracle.Head(C_IN, 0, C, theta=theta.copy(), lr=LR, momentum=MOMENTUM, dtype=np.float64)
    stride, next_key, keys, others = MIN_STRIDE, 0, [], []
    for f, (feat, T) in enumerate(frames):
        lab = oracle.teacher_labels(T)                                   # the teacher's view of every frame
        if f == next_key:
            r = oracle.train_key_frame(head, feat, lab, THRESHOLD, MAX_UPDATES)
            stride = osched.next_stride(stride, r.best_metric, THRESHOLD, MIN_STRIDE, MAX_STRIDE)
            next_key = f + stride
            keys.append((f, r.n_updates, r.best_metric, stride))
        else:                                                            # a frame the client segments on its own
            others.append((f, oracle.agreement(lab, oracle.student_mask(head, feat), C)[1]))
    return keys, others, head


def test_server_and_client_schedule_on_a_drifting_clip():
    frames = clip()
    theta = si.initial_head_params(C_IN, 0, C, 1000 + SEED)
    ref_keys, ref_others, head = oracle_loop(frames, theta)
    assert len({k[3] for k in ref_keys}) > 1 and {k[1] for k in ref_keys} >= {0, MAX_UPDATES}   # the clip exercises the rules

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        server = st.st_init_head(n_streams=1, c_in=C_IN, c_hidden=0, n_classes=C, feat_h=FH, feat_w=FW, gemm_precision=0,
                                 lr=LR, momentum=MOMENTUM, cuda_stream=stream.cuda_stream, init_params=theta)
        client = st.st_init_head(n_streams=1, c_in=C_IN, c_hidden=0, n_classes=C, feat_h=FH, feat_w=FW, gemm_precision=0,
                                 cuda_stream=stream.cuda_stream, init_params=theta)
        stride, next_key, keys, others = MIN_STRIDE, 0, [], []
        n_up, best = np.zeros(1, np.int32), np.zeros(1, np.float64)
        update = np.empty(server.n_params, np.float32)
        for f, (feat, T) in enumerate(frames):
            feat_d, T_d = torch.from_numpy(feat).cuda(), torch.from_numpy(T).cuda()
            if f == next_key:
                st.st_set_frozen_features(server, 0, feat_d)
                st.st_teacher_labels(server, 0, T_d)                      # label <- Forward(teacher, frame)
                st.st_train_key_frame(server, THRESHOLD, MAX_UPDATES, n_updates=n_up, best_metric=best)
                st.st_pack_updated_params(server, 0, update)             # (updated parameters, metric) to the client
                st.st_apply_update(client, 0, update)
                stride = st.st_next_stride(stride, float(best[0]), THRESHOLD, MIN_STRIDE, MAX_STRIDE)
                next_key = f + stride
                keys.append((f, int(n_up[0]), float(best[0]), stride))
            else:
                st.st_set_frozen_features(client, 0, feat_d)
                st.st_teacher_labels(client, 0, T_d)                      # measurement only: what the teacher would say
                others.append((f, st.st_agreement(client, 0)))
        got = np.empty(server.n_params, np.float32)
        st.st_pack_updated_params(client, 0, got)
        st.st_destroy(server)
        st.st_destroy(client)

    assert [k[0] for k in keys] == [k[0] for k in ref_keys]              # the same key frames
    assert [k[1] for k in keys] == [k[1] for k in ref_keys]              # the same number of updates on each
    assert [k[3] for k in keys] == [k[3] for k in ref_keys]              # the same strides
    np.testing.assert_allclose([k[2] for k in keys], [k[2] for k in ref_keys], atol=1e-3)
    assert [o[0] for o in others] == [o[0] for o in ref_others]
    np.testing.assert_allclose([o[1] for o in others], [o[1] for o in ref_others], atol=1e-3)
    ref = head.theta.astype(np.float64)
    assert np.linalg.norm(got - ref) <= 1e-3 * np.linalg.norm(ref)
