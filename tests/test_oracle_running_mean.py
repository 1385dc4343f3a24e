"""Pins for the oracle's Algorithm 2 server loop (side information = running mean of what was decoded so far).
It is tied to the already pinned given-vector decoder worker by worker, and to the NDQSG theorem."""
import numpy as np
import pytest

import oracle

SEED = 0x5151_AAAA_0F0F_1234


def _messages(rng, n, B, W_dqsg, W_nd, K=4, M1=4.0, bits=2, noise=0.05, alpha=1.0):
    c = rng.uniform(-0.7, 0.7, n).astype(np.float32)
    grads, msgs = [], []
    for w in range(W_dqsg + W_nd):
        g = (c + noise * rng.standard_normal(n)).astype(np.float32)
        g[::B] = 1.0
        grads.append(g)
        if w < W_dqsg:
            pk, sc = oracle.dqsg_encode(g, SEED + w, w, 7, B, 4, 9)          # Delta_1 = 1/4 as the nested fine step
            msgs.append(oracle.Msg(pk, sc, SEED + w, w, oracle.KIND_DQSG, B, 4, 9))
        else:
            pk, sc = oracle.ndqsg_encode(g, SEED + w, w, 7, B, bits, K, M1, alpha)
            msgs.append(oracle.Msg(pk, sc, SEED + w, w, oracle.KIND_NDQSG, B, bits, coarse_K=K, fine_M=M1, alpha=alpha))
    return grads, msgs


@pytest.mark.parametrize("alpha", [1.0, 0.9])
def test_running_decoder_equals_given_vector_decoder_worker_by_worker(alpha):
    rng = np.random.default_rng(1)
    n, B = 8192, 256
    grads, msgs = _messages(rng, n, B, 2, 3, alpha=alpha)
    avg, rec, qhat = oracle.decode_aggregate(msgs, n, 7, running=True, want_recon=True, want_qhat=True)
    S = np.zeros(n, dtype=np.float32)
    for w, m in enumerate(msgs):
        if m.kind == oracle.KIND_DQSG:
            r = oracle.decode_aggregate([m], n, 7)
        else:
            y = (S * (np.float32(1.0) / np.float32(w))).astype(np.float32)   # mean of the w reconstructions so far
            r = oracle.decode_aggregate([m], n, 7, side_info=y)
        assert np.array_equal(rec[w], r), f"worker {w}"
        S = (S + r).astype(np.float32)
    assert np.array_equal(avg, S / np.float32(len(msgs)))                    # the result is the mean over all W


def test_running_decoder_recovers_fine_indices_and_tracks_the_true_mean():
    rng = np.random.default_rng(2)
    n, B = 1 << 15, 1024
    grads, msgs = _messages(rng, n, B, 2, 6, noise=0.03)
    q1 = [None, None] + [oracle.ndqsg_encode(grads[w], SEED + w, w, 7, B, 2, 4, 4.0, want_q1=True)[2] for w in range(2, 8)]
    avg, rec, qhat = oracle.decode_aggregate(msgs, n, 7, running=True, want_recon=True, want_qhat=True)
    for w in range(2, 8):
        assert (qhat[w] == q1[w]).mean() > 0.999        # z = g_w - g_bar is far inside (Delta2 - Delta1)/2 = 0.375
    true = np.mean(grads, axis=0)
    err = avg - true
    assert np.abs(err).max() < 0.125 + 1e-3            # every worker is within Delta_1/2 = 1/8 of its gradient
    assert err.std() < (0.25 / np.sqrt(12)) / np.sqrt(8) * 1.2


def test_running_decoder_needs_a_dqsg_message_first():
    rng = np.random.default_rng(3)
    grads, msgs = _messages(rng, 512, 64, 1, 1)
    with pytest.raises(ValueError):
        oracle.decode_aggregate(msgs[::-1], 512, 7, running=True)
    out = oracle.decode_aggregate(msgs[:1], 512, 7, running=True)            # DQSG only: plain Algorithm 1
    assert np.array_equal(out, oracle.decode_aggregate(msgs[:1], 512, 7))
