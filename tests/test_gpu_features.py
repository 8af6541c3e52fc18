"""On-device saliency features (Eq. 14-17) against the fp64 oracle definitions."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

BITS = np.array([2, 4, 8, 16], np.uint8)


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_04722_b200 import build
    build.build()
    import gpu_util
    return gpu_util


def _features(gu, logits, token_ids, counts, total, observed, attn_var):
    import torch
    from paper_2604_04722_b200 import binding as kq
    n, vocab = logits.shape
    ld = torch.from_numpy(np.ascontiguousarray(logits)).to(gu.DEV)
    ids = torch.from_numpy(token_ids.astype(np.int32)).to(gu.DEV)
    cd = torch.from_numpy(counts.astype(np.int64)).to(torch.int32).to(gu.DEV)
    av = torch.from_numpy(attn_var.astype(np.float32)).to(gu.DEV) if attn_var is not None else None
    feats = torch.zeros((n, 4), dtype=torch.float32, device=gu.DEV)
    kq.kvq_token_features(ld, logits.dtype == np.float32, n, vocab, ids, cd, total, observed, av, feats)
    torch.cuda.synchronize()
    return feats.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("vocab,dtype,scale", [(49152, np.float16, 3.0), (49152, np.float32, 8.0), (1001, np.float16, 2.0),
                                               (1001, np.float32, 0.1), (8, np.float32, 1.0), (70000, np.float16, 12.0)])
def test_token_features_match_the_definitions(gu, oracle, vocab, dtype, scale):
    rng = np.random.default_rng(vocab + int(scale * 10))
    n = 37
    logits = (rng.standard_normal((n, vocab)) * scale).astype(dtype)
    logits[3] = dtype(1.25)                                   # uniform distribution: H = log |V|, C = 1/|V|
    logits[4] = dtype(-30.0)
    logits[4, vocab // 2] = dtype(40.0)                       # one-hot: H ~ 0, C ~ 1
    token_ids = rng.integers(0, vocab, size=n)
    counts = rng.integers(0, 5000, size=vocab)
    counts[token_ids[0]] = 0
    total, observed = int(counts.sum()), int((counts > 0).sum())
    attn_var = rng.random(n) * 1e-3
    got = _features(gu, logits, token_ids, counts, total, observed, attn_var)
    H = oracle.token_entropy(logits)
    C = oracle.token_confidence(logits)
    R = oracle.token_rarity(token_ids, counts, total, observed)
    assert np.all(np.abs(got[:, 0] - H) <= 2e-4 + 2e-4 * np.abs(H)), np.abs(got[:, 0] - H).max()
    assert np.all(np.abs(got[:, 1] - R) <= 1e-5 * np.abs(R) + 1e-6)
    assert np.array_equal(got[:, 2].astype(np.float32), attn_var.astype(np.float32))
    assert np.all(np.abs(got[:, 3] - C) <= 1e-3 * C + 1e-9)
    no_var = _features(gu, logits[:2], token_ids[:2], counts, total, observed, None)
    assert np.all(no_var[:, 2] == 0.0) and np.allclose(no_var[:, [0, 1, 3]], got[:2][:, [0, 1, 3]])


@pytest.mark.parametrize("vocab,dtype", [(49152, np.float16), (1001, np.float32), (4096, np.float32)])
def test_token_features_with_masked_logits(gu, oracle, vocab, dtype):
    """Vocabulary entries masked with -inf (p = 0, so p log p = 0 in Eq. 14) leave entropy and confidence
    finite and equal to those of the unmasked entries: at the start of a row, in whole 8-element groups,
    scattered, and all but one entry."""
    rng = np.random.default_rng(vocab)
    n = 9
    logits = (rng.standard_normal((n, vocab)) * 3).astype(dtype)
    logits[0, :16] = -np.inf                                  # the row starts with masked groups
    logits[1, ::3] = -np.inf                                  # scattered
    logits[2, vocab // 2:] = -np.inf                          # a masked tail
    logits[3, :] = -np.inf
    logits[3, 5] = dtype(0.75)                                # a single survivor: H = 0, C = 1
    logits[4, :vocab - 3] = -np.inf                           # survivors only in the last group
    token_ids = rng.integers(0, vocab, size=n)
    counts = rng.integers(0, 50, size=vocab)
    got = _features(gu, logits, token_ids, counts, int(counts.sum()), int((counts > 0).sum()), None)
    with np.errstate(invalid="ignore"):
        H = oracle.token_entropy(logits)
        C = oracle.token_confidence(logits)
    assert np.all(np.isfinite(got))
    assert np.all(np.abs(got[:, 0] - H) <= 2e-4 + 2e-4 * np.abs(H)), (got[:, 0], H)
    assert np.all(np.abs(got[:, 3] - C) <= 1e-3 * C + 1e-9)
    assert got[3, 0] == 0.0 and got[3, 3] == 1.0


@pytest.mark.parametrize("n,splits", [(1, 0), (17, 0), (700, 0), (700, 7), (3000, 0)])
def test_attention_variance_of_the_decode_step(gu, oracle, n, splits):
    """kvq_decode_attn_var: V = mean over heads of the variance of the attention weights over the cached
    tokens (Eq. 16), from the sums of squared weights the decode kernel keeps; the attention output is the
    one kvq_decode_attn gives."""
    import torch
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(n + splits)
    B, Hq, H = 3, 6, 2
    bits = BITS[rng.choice(4, size=(B, n), p=[.4, .3, .2, .1])]
    K = (rng.standard_normal((B, n, H, 64)) * 1.5).astype(np.float16)
    V = (rng.standard_normal((B, n, H, 64)) * 1.5).astype(np.float16)
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    oc = oracle.OracleCache(B, Hq, H)
    oc.append(K, V, bits)
    want = oracle.attention_variance(oc.decode_probs(Q))
    with gu.GpuCache(1, B, Hq, H, n) as g:
        g.append(0, K, V, bits)
        kq.kvq_set_splits(g.ctx, splits)
        Qd = gu.dev(Q.view(np.uint16))
        O = torch.zeros_like(Qd)
        var = torch.zeros(B, dtype=torch.float32, device=gu.DEV)
        kq.kvq_decode_attn_var(g.ctx, 0, Qd, O, var)
        torch.cuda.synchronize()
        got = var.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - want) <= 2e-3 * np.abs(want) + 1e-7 / n), (got, want)
        gu.assert_attention_close(O.cpu().numpy().view(np.uint16), oc.decode_attn(Q), "output of the variance call")
        assert np.array_equal(O.cpu().numpy().view(np.uint16), g.decode(0, Q))
