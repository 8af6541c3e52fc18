"""The arena of packed rows: blocks are taken when an append first reaches them, the memory in use
follows the stored row bytes (the footprint side of the paper's claim, Section 3.1 / Eq. 10-11),
block borders are invisible to the store's content and to attention, and running out of blocks is
reported, not faulted."""
import numpy as np
import pytest

from paper_2604_04722_b200 import synth

pytestmark = pytest.mark.gpu

BITS = np.array([2, 4, 8, 16], np.uint8)
BLOCK_TOKENS = {2: 1600, 4: 880, 8: 480, 16: 256}      # tokens of one stream that fit a 64 KB block
ROW_BYTES = {2: 40, 4: 72, 8: 136, 16: 256}


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_04722_b200 import build
    build.build()
    import gpu_util
    return gpu_util


def _expected_blocks(counts, kv_heads):
    """Blocks in use for per-sequence class counts [batch][4]: one stream per (sequence, head, class)."""
    total = 0
    for row in counts:
        for k, b in enumerate((2, 4, 8, 16)):
            total += kv_heads * (-(-int(row[k]) // BLOCK_TOKENS[b]))
    return total


def _kv(rng, B, n, H):
    K = (rng.standard_normal((B, n, H, 64)) * 1.5).astype(np.float16)
    V = (rng.standard_normal((B, n, H, 64)) * 1.5).astype(np.float16)
    return K, V


@pytest.mark.parametrize("bt,n", [(2, 3700), (4, 2000), (8, 1100), (16, 600)])
def test_streams_that_span_several_blocks(gu, oracle, bt, n):
    """Uniform precision long enough that every stream crosses block borders: the store is bit-exact,
    attention within tolerance, and exactly ceil(n / tokens-per-block) blocks per stream are in use."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(bt * 1000 + n)
    B, Hq, H = 2, 4, 2
    K, V = _kv(rng, B, n, H)
    bits = np.full((B, n), bt, np.uint8)
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    oc = oracle.OracleCache(B, Hq, H)
    oc.append(K, V, bits)
    with gu.GpuCache(1, B, Hq, H, n) as g:
        g.append(0, K, V, bits)
        used, total, block_bytes = kq.kvq_arena_usage(g.ctx)
        assert block_bytes == 65536
        assert used == B * H * (-(-n // BLOCK_TOKENS[bt]))
        gu.assert_store_equals_oracle(g, 0, oc, pos0=n - 300, n=300)
        gu.assert_store_equals_oracle(g, 0, oc, pos0=BLOCK_TOKENS[bt] - 40, n=80)     # around the first border
        for splits in (0, 1, 5):
            kq.kvq_set_splits(g.ctx, splits)
            gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "bits=%d splits=%d" % (bt, splits))


def test_usage_follows_prefill_chunk_appends_and_decode_steps(gu, oracle):
    """Mixed precisions appended three ways (a multi-chunk prefill, a one-chunk append, single-token
    steps): after each, the blocks in use are exactly those the pool fills call for, on both layers."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(77)
    B, Hq, H, L = 3, 6, 3, 2
    pieces = [1900, 200] + [1] * 40
    n_total = sum(pieces)
    ocs = [oracle.OracleCache(B, Hq, H) for _ in range(L)]
    with gu.GpuCache(L, B, Hq, H, n_total) as g:
        for i, n in enumerate(pieces):
            for layer in range(L):
                K, V = _kv(rng, B, n, H)
                # a skewed mix so that the 16-bit streams cross their 256-token border during the steps
                bits = BITS[rng.choice(4, size=(B, n), p=[.35, .25, .25, .15])]
                ocs[layer].append(K, V, bits)
                g.append(layer, K, V, bits)
            if i in (0, 1, len(pieces) - 1):
                want = sum(_expected_blocks(kq.kvq_stats(g.ctx, layer, B)[0], H) for layer in range(L))
                assert kq.kvq_arena_usage(g.ctx)[0] == want
        for layer in range(L):
            gu.assert_store_equals_oracle(g, layer, ocs[layer])
            Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
            gu.assert_attention_close(g.decode(layer, Q), ocs[layer].decode_attn(Q), "layer %d" % layer)
        assert kq.kvq_device_status(g.ctx) == 0


def test_a_budget_near_the_stored_bytes_is_enough(gu, oracle):
    """kvq_create_arena with a budget of the stored row bytes plus one block of slack per stream: the
    cache works, and what is in use stays within that budget -- far below the worst-case 504 bytes per
    token and head that kvq_create reserves, and below the 256 bytes of an fp16 cache."""
    import torch
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(5)
    B, Hq, H, n = 4, 8, 4, 6000
    mix = [.5, .3, .15, .05]
    bits = BITS[rng.choice(4, size=(B, n), p=mix)]
    K, V = _kv(rng, B, n, H)
    stored = sum(ROW_BYTES[int(b)] for b in bits.ravel()) * H
    budget = stored + (B * H * 4 + 1) * 65536
    ctx = kq.kvq_create_arena(1, Hq, H, 64, n, B, budget)
    try:
        Kd, Vd, bd = gu.dev(K.view(np.uint16)), gu.dev(V.view(np.uint16)), gu.dev(bits)
        kq.kvq_append(ctx, 0, Kd, Vd, bd, n)
        used, total, block_bytes = kq.kvq_arena_usage(ctx)
        assert total == budget // 65536 - 1
        assert used * block_bytes <= budget
        assert used * block_bytes < 0.5 * (B * H * n * 256)           # less than half of an fp16 cache here
        assert kq.kvq_device_status(ctx) == 0
        _, resident, ebits = kq.kvq_stats(ctx, 0, B)
        assert resident == stored and abs(ebits - float(np.mean(bits.astype(np.float64)))) < 1e-9
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        Qd = gu.dev(Q.view(np.uint16))
        O = torch.zeros_like(Qd)
        kq.kvq_decode_attn(ctx, 0, Qd, O)
        torch.cuda.synchronize()
        seqs = [1]
        oc = oracle.OracleCache(len(seqs), Hq, H)
        oc.append(K[seqs], V[seqs], bits[seqs])
        gu.assert_attention_close(O.cpu().numpy().view(np.uint16)[seqs], oc.decode_attn(Q[seqs]), "budgeted arena")
    finally:
        kq.kvq_destroy(ctx)


def test_running_out_of_blocks_is_flagged_not_faulted(gu):
    """Six blocks cannot hold 2 sequences x 2 heads x 2 tensors of 600 fp16 tokens (12 needed): the append
    sets KVQ_FLAG_ARENA_FULL; after kvq_reset a smaller append fits and raises nothing."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(6)
    B, Hq, H, n = 2, 2, 2, 600
    K, V = _kv(rng, B, n, H)
    ctx = kq.kvq_create_arena(1, Hq, H, 64, n, B, 7 * 65536)             # block 0 is never handed out: six usable
    try:
        Kd, Vd = gu.dev(K.view(np.uint16)), gu.dev(V.view(np.uint16))
        kq.kvq_append(ctx, 0, Kd, Vd, gu.dev(np.full((B, n), 16, np.uint8)), n)
        assert kq.kvq_device_status(ctx) & 4
        assert kq.kvq_arena_usage(ctx)[0] == 6
        kq.kvq_reset(ctx)
        kq.kvq_append(ctx, 0, Kd[:, :200].contiguous(), Vd[:, :200].contiguous(),
                      gu.dev(np.full((B, 200), 16, np.uint8)), 200)
        assert kq.kvq_device_status(ctx) == 0
        assert kq.kvq_arena_usage(ctx)[0] == B * H
    finally:
        kq.kvq_destroy(ctx)


def test_recycled_blocks_do_not_leak_into_attention(gu, oracle):
    """Blocks go back to the arena on kvq_reset and come back holding another stream's bytes.  Fill the
    cache with fp16 rows of huge values, reset, then append a mix whose 8-bit tokens all sit in the
    first chunk of a multi-chunk append (their last tile stays partly filled): the unused slots of every
    last tile must carry no weight, whatever the recycled blocks held."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(8)
    B, Hq, H, n = 2, 4, 2, 1000
    big = np.full((B, n, H, 64), 60000.0, np.float16)
    big[..., ::3] = np.float16("inf")
    with gu.GpuCache(1, B, Hq, H, n) as g:
        g.append(0, big, big, np.full((B, n), 16, np.uint8))
        for steps in (0, 3):
            kq.kvq_reset(g.ctx)
            K, V = _kv(rng, B, n, H)
            bits = BITS[rng.choice(2, size=(B, n))]                   # 2- and 4-bit ...
            bits[:, 5:42:3] = 8                                        # ... and a few 8-bit tokens early on
            oc = oracle.OracleCache(B, Hq, H)
            oc.append(K[:, :n - steps], V[:, :n - steps], bits[:, :n - steps])
            g.append(0, K[:, :n - steps], V[:, :n - steps], bits[:, :n - steps])
            for i in range(n - steps, n):                              # single-token appends open tiles too
                oc.append(K[:, i:i + 1], V[:, i:i + 1], bits[:, i:i + 1])
                g.append(0, K[:, i:i + 1], V[:, i:i + 1], bits[:, i:i + 1])
            Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
            gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "after reset, %d steps" % steps)
