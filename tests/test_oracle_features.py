"""Pins of the oracle's token-level saliency features (Eq. 14-17): closed forms, limits and library routines."""
import math

import numpy as np


def test_entropy_closed_forms_and_library_routine(oracle):
    V = 1000
    assert abs(oracle.token_entropy(np.zeros((1, V)))[0] - math.log(V)) < 1e-12            # uniform -> log |V|
    z = np.full((1, V), -1e4)
    z[0, 7] = 0.0
    assert oracle.token_entropy(z)[0] < 1e-12                                                  # one-hot -> 0
    # two equal peaks and nothing else -> log 2; shifting all logits changes nothing
    z = np.full((1, V), -1e4)
    z[0, [3, 9]] = 5.0
    assert abs(oracle.token_entropy(z)[0] - math.log(2)) < 1e-12
    rng = np.random.default_rng(0)
    z = rng.standard_normal((6, 777)) * 4
    assert np.allclose(oracle.token_entropy(z), oracle.token_entropy(z + 123.0), atol=1e-12)
    from scipy.stats import entropy
    from scipy.special import softmax
    assert np.allclose(oracle.token_entropy(z), entropy(softmax(z, axis=1), axis=1), atol=1e-12)
    # bounds: 0 <= H <= log V
    h = oracle.token_entropy(z)
    assert np.all(h >= 0) and np.all(h <= math.log(777) + 1e-12)


def test_masked_logits_add_nothing_to_the_entropy(oracle):
    """p log p is 0 at p = 0 (Eq. 14): a vocabulary entry masked with -inf drops out, so the entropy is that of
    the remaining entries; the same for the confidence."""
    rng = np.random.default_rng(3)
    z = rng.standard_normal((4, 200)) * 2
    masked = np.concatenate([np.full((4, 30), -np.inf), z, np.full((4, 7), -np.inf)], axis=1)
    with np.errstate(invalid="ignore"):
        assert np.allclose(oracle.token_entropy(masked), oracle.token_entropy(z), atol=1e-12)
        assert np.allclose(oracle.token_confidence(masked), oracle.token_confidence(z), atol=1e-15)
    one = np.full((1, 64), -np.inf)
    one[0, 11] = 2.5
    assert oracle.token_entropy(one)[0] == 0.0 and oracle.token_confidence(one)[0] == 1.0


def test_confidence_is_the_largest_probability(oracle):
    V = 50
    assert abs(oracle.token_confidence(np.zeros((1, V)))[0] - 1.0 / V) < 1e-15
    z = np.zeros((1, V))
    z[0, 4] = math.log(3.0)                      # p = 3 / (V - 1 + 3)
    assert abs(oracle.token_confidence(z)[0] - 3.0 / (V + 2)) < 1e-15
    from scipy.special import softmax
    z = np.random.default_rng(1).standard_normal((5, 300)) * 3
    assert np.allclose(oracle.token_confidence(z), softmax(z, axis=1).max(axis=1), atol=1e-15)


def test_rarity_is_smoothed_self_information(oracle):
    counts = np.array([0, 9, 99, 4], dtype=np.uint32)
    total, observed = 112, 3
    r = oracle.token_rarity([0, 1, 2, 3, 1], counts, total, observed)
    want = [-math.log((c + 1) / (total + observed + 1)) for c in (0, 9, 99, 4, 9)]
    assert np.allclose(r, want, atol=1e-15)
    assert r[0] > r[3] > r[1] > r[2]             # rarer tokens score higher
    # an unseen token in an empty stream: -log(1 / 1) = 0
    assert oracle.token_rarity([2], np.zeros(5, np.uint32), 0, 0)[0] == 0.0


def test_attention_variance_closed_forms(oracle):
    n, h = 40, 3
    uniform = np.full((1, h, n), 1.0 / n)
    assert abs(oracle.attention_variance(uniform)[0]) < 1e-18
    onehot = np.zeros((1, h, n))
    onehot[0, :, 5] = 1.0
    assert abs(oracle.attention_variance(onehot)[0] - (1.0 / n) * (1.0 - 1.0 / n)) < 1e-15   # E[a^2] - E[a]^2
    mixed = np.concatenate([uniform[:, :1], onehot[:, :2]], axis=1)                           # mean over heads
    assert abs(oracle.attention_variance(mixed)[0] - (2.0 / 3.0) * (1.0 / n) * (1.0 - 1.0 / n)) < 1e-15
    # since the weights sum to one: Var = sum a^2 / n - 1 / n^2
    a = np.random.default_rng(2).random((2, h, n))
    a /= a.sum(axis=2, keepdims=True)
    assert np.allclose(oracle.attention_variance(a), ((a ** 2).sum(axis=2) / n - 1.0 / n ** 2).mean(axis=1), atol=1e-15)


def test_attention_weights_of_the_cache_sum_to_one_and_reproduce_the_output(oracle):
    rng = np.random.default_rng(3)
    B, Hq, H, n = 2, 4, 2, 70
    K = rng.standard_normal((B, n, H, 64)).astype(np.float16)
    V = rng.standard_normal((B, n, H, 64)).astype(np.float16)
    bits = np.array([2, 4, 8, 16], np.uint8)[rng.choice(4, size=(B, n))]
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    oc = oracle.OracleCache(B, Hq, H)
    oc.append(K, V, bits)
    p = oc.decode_probs(Q)
    assert p.shape == (B, Hq, n) and np.allclose(p.sum(axis=2), 1.0, atol=1e-12) and np.all(p >= 0)
    # the weights times the dequantized value rows give the attention output
    _, out64 = oc.decode_attn(Q, want64=True)
    for b in range(B):
        for h in range(Hq):
            vhat = np.stack([oracle.dequantize_row(oc.vc[b, t, h // 2], oc.vm[b, t, h // 2], 64, int(bits[b, t]))
                             for t in range(n)]).astype(np.float64)
            assert np.allclose(p[b, h] @ vhat, out64[b, h], atol=1e-10)
