"""Pins for the oracle's controller (Eq. 19-23) -- CPU only."""
import numpy as np

from paper_2604_04722_b200 import synth


def _zeros(hidden):
    return [np.zeros((hidden, 4), np.float32), np.zeros(hidden, np.float32),
            np.zeros((hidden, hidden), np.float32), np.zeros(hidden, np.float32),
            np.zeros((4, hidden), np.float32), np.zeros(4, np.float32)]


def test_identity_weights_select_the_largest_feature(oracle):
    """W1, W2, W3 copy the four non-negative features through both ReLUs, so the logits are the
    features and the class is the position of the largest one; IndexToBit maps it to {2,4,8,16}."""
    hidden = 8
    W1, b1, W2, b2, W3, b3 = _zeros(hidden)
    for k in range(4):
        W1[k, k] = 1
        W2[k, k] = 1
        W3[k, k] = 1
    rng = np.random.default_rng(0)
    feats = rng.random((500, 4)).astype(np.float32)
    bits, logits, gap = oracle.select_bits(feats, hidden, W1, b1, W2, b2, W3, b3)
    assert np.array_equal(logits, feats)
    assert np.array_equal(bits, np.array([2, 4, 8, 16], np.uint8)[feats.argmax(1)])
    srt = np.sort(feats, 1)
    assert np.array_equal(gap, srt[:, 3] - srt[:, 2])
    # negative features are cut by the first ReLU
    neg = -feats
    bits, logits, _ = oracle.select_bits(neg, hidden, W1, b1, W2, b2, W3, b3)
    assert not logits.any() and np.all(bits == 2)


def test_ties_go_to_the_lowest_class_and_nan_to_fp16(oracle):
    hidden = 4
    w = _zeros(hidden)
    feats = np.ones((3, 4), np.float32)
    bits, logits, gap = oracle.select_bits(feats, hidden, *w)
    assert np.all(bits == 2) and not logits.any() and not gap.any()
    w[5][:] = [0, 0, 0, 1]                       # b3 favours class 3
    assert np.all(oracle.select_bits(feats, hidden, *w)[0] == 16)
    w[5][:] = [0, 5, 5, 1]                       # two equal maxima: the first wins
    assert np.all(oracle.select_bits(feats, hidden, *w)[0] == 4)
    w[5][:] = [9, np.nan, 0, 0]
    bits, _, gap = oracle.select_bits(feats, hidden, *w)
    assert np.all(bits == 16) and np.all(np.isnan(gap))


def test_multiply_and_add_round_separately_in_ascending_order(oracle):
    """fp32, product rounded, then sum rounded, i ascending.

    (1+2^-12)^2 = 1 + 2^-11 + 2^-24 rounds to 1 + 2^-11 in fp32 (tie to even); with the bias
    -(1+2^-11) the unfused result is exactly 0, a fused multiply-add would give 2^-24.
    The hidden value feeds logit 1; logits 2 and 3 are -1.  0 -> tie -> class 0; 2^-24 -> class 1.
    """
    hidden = 4
    W1, b1, W2, b2, W3, b3 = _zeros(hidden)
    a = np.float32(1 + 2.0 ** -12)
    W1[0, 0] = a
    b1[0] = -np.float32(1 + 2.0 ** -11)
    W2[0, 0] = 1
    W3[1, 0] = 1
    b3[:] = [0, 0, -1, -1]
    feats = np.array([[a, 0, 0, 0]], np.float32)
    bits, logits, _ = oracle.select_bits(feats, hidden, W1, b1, W2, b2, W3, b3)
    assert logits[0, 1] == 0.0 and bits[0] == 2
    # ascending accumulation: 1e8 + 3 + 3 + 3 stays 1e8 (each +3 is below half an ulp of 8),
    # while adding the terms first would reach 1e8 + 8.
    W1, b1, W2, b2, W3, b3 = _zeros(hidden)
    W1[0, :3] = 3
    b1[0] = 1e8
    W2[0, 0] = 1
    W3[0, 0] = 1
    feats = np.array([[1, 1, 1, 0]], np.float32)
    _, logits, _ = oracle.select_bits(feats, hidden, W1, b1, W2, b2, W3, b3)
    assert logits[0, 0] == np.float32(1e8)


def _mlp_fp64(feats, cw):
    h1 = np.maximum(feats.astype(np.float64) @ cw.W1.astype(np.float64).T + cw.b1, 0)
    h2 = np.maximum(h1 @ cw.W2.astype(np.float64).T + cw.b2, 0)
    return h2 @ cw.W3.astype(np.float64).T + cw.b3


def test_random_controller_against_fp64_matrix_products(oracle):
    for hidden, seed in ((32, 0), (32, 1), (128, 2)):
        cw = synth.controller_weights(seed, hidden)
        feats = synth.features(seed, 0, 0, 4000)
        bits, logits, gap = oracle.select_bits(feats, hidden, *cw.as_tuple())
        ref = _mlp_fp64(feats, cw)
        assert np.allclose(logits, ref, rtol=1e-4, atol=1e-4)
        clear = gap > 1e-4
        assert clear.mean() > 0.9
        want = np.array([2, 4, 8, 16], np.uint8)[ref.argmax(1)]
        assert np.array_equal(bits[clear], want[clear])
        # Eq. 22-23: argmax of the softmax probabilities equals argmax of the logits
        e = np.exp(ref - ref.max(1, keepdims=True))
        p = e / e.sum(1, keepdims=True)
        assert np.array_equal(p.argmax(1)[clear], ref.argmax(1)[clear])


def test_feature_and_weight_recipe():
    f = synth.features(0, 0, 0, 20000)
    assert f.dtype == np.float32 and f.shape == (20000, 4)
    assert 0 <= f[:, 0].min() and f[:, 0].max() <= 1 and np.median(f[:, 0]) < 0.05   # Zipf: mass at low ranks
    assert 0 <= f[:, 1].min() and f[:, 1].max() < 1
    assert abs(np.log(f[:, 2]).mean() + 2) < 0.05
    assert f[:, 3].max() <= np.log(49152) and f[:, 3].min() >= 0
    cw = synth.controller_weights(0, 32)
    assert np.abs(cw.W2).max() <= np.sqrt(6 / 32) and np.abs(cw.b2).max() <= 1 / np.sqrt(32)
    assert np.array_equal(synth.features(3, 1, 7, 50), synth.features(3, 1, 7, 50))
