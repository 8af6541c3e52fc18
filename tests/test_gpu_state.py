"""Snapshots: kvq_save_state / kvq_load_state.  A cache restored from a snapshot, into the same handle or a fresh
one, continues exactly like the one the snapshot was taken from."""
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


def _kv(rng, B, n, H):
    K = (rng.standard_normal((B, n, H, 64)) * 2).astype(np.float16)
    V = rng.standard_normal((B, n, H, 64)).astype(np.float16)
    return K, V


@pytest.mark.parametrize("groups", [1, 2])
def test_restore_and_continue(gu, oracle, groups):
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(40 + groups)
    L, B, Hq, H = 2, 3, 4, 2
    lens = [500, 123, 0]
    oc = [oracle.OracleCache(1, Hq, H) if groups == 1 else oracle.GroupedOracleCache(1, Hq, H, 2) for _ in range(B)]

    def add(g, K, V, bits, ls=None):
        if ls is None:
            g.append(1, K, V, bits)
        else:
            kq.kvq_append_ragged(g.ctx, 1, gu.dev(K.view(np.uint16)), gu.dev(V.view(np.uint16)), gu.dev(bits), None, K.shape[1], ls)

    K0, V0 = _kv(rng, B, 500, H)
    b0 = BITS[rng.choice(4, size=(B, 500), p=[.4, .3, .2, .1])]
    later = []
    for n in (1, 40, 1):
        K, V = _kv(rng, B, n, H)
        later.append((K, V, BITS[rng.choice(4, size=(B, n))]))
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)

    with gu.GpuCache(L, B, Hq, H, 600, scale_groups=groups) as g:
        add(g, K0, V0, b0, lens)
        blob = kq.kvq_save_state(g.ctx)
        assert blob.size < 3 * 2 ** 20                  # rows in use, not the worst-case arena
        for K, V, bits in later:
            add(g, K, V, bits)
        want_out = g.decode(1, Q)
        want_store = g.export(1, 0, 42)                 # every sequence holds at least 42 tokens now
        # back to the snapshot in the same handle
        kq.kvq_load_state(g.ctx, blob)
        assert kq.kvq_seq_lens(g.ctx, 1, B).tolist() == lens and kq.kvq_seq_len(g.ctx, 0) == 0
        for K, V, bits in later:
            add(g, K, V, bits)
        assert np.array_equal(g.decode(1, Q), want_out)
    # and in a fresh handle with a smaller arena
    with gu.GpuCache(L, B, Hq, H, 600, scale_groups=groups, arena_bytes=64 * 65536) as g2:
        kq.kvq_load_state(g2.ctx, blob)
        for K, V, bits in later:
            add(g2, K, V, bits)
        assert np.array_equal(g2.decode(1, Q), want_out)
        for a, b in zip(g2.export(1, 0, 42), want_store):
            assert np.array_equal(a, b)
        # against the oracle as well
        for b in range(B):
            if lens[b]:
                oc[b].append(K0[b:b + 1, :lens[b]], V0[b:b + 1, :lens[b]], b0[b:b + 1, :lens[b]])
            for K, V, bits in later:
                oc[b].append(K[b:b + 1], V[b:b + 1], bits[b:b + 1])
            gu.assert_attention_close(want_out[b:b + 1], oc[b].decode_attn(Q[b:b + 1]), "sequence %d" % b)


def test_snapshots_of_other_shapes_are_refused(gu):
    from paper_2604_04722_b200 import binding as kq
    with gu.GpuCache(1, 1, 2, 2, 32) as a, gu.GpuCache(1, 1, 2, 1, 32) as b, gu.GpuCache(1, 1, 2, 2, 32, scale_groups=2) as c:
        blob = kq.kvq_save_state(a.ctx)
        L = kq.lib()
        assert L.kvq_load_state(b.ctx, blob.ctypes.data, blob.size) == kq.KVQ_ERR_ARG
        assert L.kvq_load_state(c.ctx, blob.ctypes.data, blob.size) == kq.KVQ_ERR_ARG
        assert L.kvq_load_state(a.ctx, blob.ctypes.data, blob.size - 1) == kq.KVQ_ERR_ARG
        bad = blob.copy()
        bad[0] ^= 0xff
        assert L.kvq_load_state(a.ctx, bad.ctypes.data, bad.size) == kq.KVQ_ERR_ARG
        assert L.kvq_save_state(a.ctx, blob.ctypes.data, blob.size - 1) == kq.KVQ_ERR_ARG
        kq.kvq_load_state(a.ctx, blob)


def test_a_snapshot_that_points_outside_the_cache_is_refused(gu):
    """Block ids, index words, fills and lengths of a blob are checked on the host before anything is loaded."""
    import struct
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(2)
    B, Hq, H, n = 1, 2, 2, 40
    with gu.GpuCache(1, B, Hq, H, 64) as g:
        K, V = _kv(rng, B, n, H)
        g.append(0, K, V, BITS[rng.choice(4, size=(B, n))])
        blob = kq.kvq_save_state(g.ctx)
        head = struct.calcsize("<II6iII4Q")
        used = struct.unpack_from("<I", blob, 4 * 9)[0]
        table_bytes, index_bytes, counts_bytes, total = struct.unpack_from("<4Q", blob, head - 32)
        assert total == blob.size
        ints = 1 * 3 + 1 * B
        table_at = head + 4 * ints + (used + 1) * 65536
        index_at = table_at + table_bytes
        counts_at = index_at + index_bytes
        L = kq.lib()

        def refused(at, value):
            bad = blob.copy()
            bad[at:at + 4] = np.frombuffer(struct.pack("<I", value), np.uint8)
            return L.kvq_load_state(g.ctx, bad.ctypes.data, bad.size) == kq.KVQ_ERR_ARG

        assert refused(table_at, used + 1)              # a block that was never handed out
        assert refused(index_at, (1 << 30) | 64)        # a slot beyond max_ctx
        assert refused(counts_at, 1000)                 # a pool fill that does not add up
        assert refused(head + 4, 65)                    # a sequence longer than max_ctx
        assert refused(head, 39)                        # longest length out of step with the lengths

        # header fields that only have to be consistent with each other to pass a naive check: sizes that are
        # not this handle's, and a block count that wraps around in 32-bit arithmetic
        def header_refused(**fields):
            bad = blob.copy()
            names = ["magic", "version", "layers", "q_heads", "kv_heads", "max_ctx", "batch", "groups", "arena_blocks",
                     "blocks_used", "table_bytes", "index_bytes", "counts_bytes", "total_bytes"]
            vals = dict(zip(names, struct.unpack_from("<II6iII4Q", bad, 0)))
            vals.update(fields)
            struct.pack_into("<II6iII4Q", bad, 0, *[vals[k] for k in names])
            return L.kvq_load_state(g.ctx, bad.ctypes.data, bad.size) == kq.KVQ_ERR_ARG

        assert header_refused(index_bytes=index_bytes + 4096, counts_bytes=counts_bytes)                 # total no longer adds up
        assert header_refused(index_bytes=index_bytes + 4096, total_bytes=total + 4096)                  # consistent, but too large
        assert header_refused(index_bytes=index_bytes - 64, counts_bytes=counts_bytes + 64)              # consistent, shifted
        assert header_refused(counts_bytes=counts_bytes - 16, total_bytes=total - 16)                    # a short fill table
        assert header_refused(blocks_used=0xffffffff)                                                    # + 1 wraps to 0
        assert header_refused(blocks_used=0xffffffff, total_bytes=total - (used + 1) * 65536)            # ... consistently
        kq.kvq_load_state(g.ctx, blob)                  # the untouched blob still loads


def test_snapshot_after_a_reset(gu):
    """After kvq_reset the block tables still hold ids from before; they are beyond the fills, are not part of the
    state, and must not make a snapshot unloadable (also not in a handle with a smaller arena)."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(6)
    B, Hq, H = 2, 2, 2
    with gu.GpuCache(1, B, Hq, H, 1200) as g:
        K, V = _kv(rng, B, 1200, H)
        g.append(0, K, V, BITS[rng.choice(4, size=(B, 1200))])      # several blocks per stream
        kq.kvq_reset(g.ctx)
        K, V = _kv(rng, B, 30, H)
        bits = BITS[rng.choice(4, size=(B, 30))]
        g.append(0, K, V, bits)
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        want = g.decode(0, Q)
        blob = kq.kvq_save_state(g.ctx)
        kq.kvq_load_state(g.ctx, blob)
        assert np.array_equal(g.decode(0, Q), want)
    with gu.GpuCache(1, B, Hq, H, 1200, arena_bytes=40 * 65536) as g2:
        kq.kvq_load_state(g2.ctx, blob)
        assert np.array_equal(g2.decode(0, Q), want)
