"""kvq_create_in: a cache whose device buffers all lie inside one allocation of the caller (here a torch
tensor).  Same results as a cache that allocates for itself, nothing written outside the workspace, nothing
freed by kvq_destroy."""
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


@pytest.mark.parametrize("groups,arena_blocks", [(1, 0), (2, 0), (1, 40)])
def test_cache_in_a_caller_owned_workspace(gu, oracle, groups, arena_blocks):
    import torch
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(3 + groups + arena_blocks)
    L, B, Hq, H, n = 2, 2, 4, 2, 300
    shape = (L, Hq, H, 64, n + 4, B)
    need = kq.kvq_workspace_bytes(*shape, arena_blocks * 65536, groups)
    assert need > 0 and need % 256 == 0
    guard = 4096
    buf = torch.full((need + 2 * guard,), 0xA5, dtype=torch.uint8, device=gu.DEV)
    ws = buf[guard:guard + need]
    assert ws.data_ptr() % 256 == 0
    with pytest.raises(kq.KvqError):                   # one byte short
        kq.kvq_create_in(*shape, arena_blocks * 65536, groups, ws, need - 1)
    import ctypes
    handle = ctypes.c_void_p()
    assert kq.lib().kvq_create_in(ctypes.byref(handle), *shape, 0, groups, ws.data_ptr() + 16, need) == kq.KVQ_ERR_ARG
    host = torch.zeros(need + 256, dtype=torch.uint8)  # host memory is not a workspace
    host_ptr = (host.data_ptr() + 255) & ~255
    assert kq.lib().kvq_create_in(ctypes.byref(handle), *shape, 0, groups, host_ptr, need) == kq.KVQ_ERR_ARG
    ctx = kq.kvq_create_in(*shape, arena_blocks * 65536, groups, ws, need)
    oc = oracle.OracleCache(B, Hq, H) if groups == 1 else oracle.GroupedOracleCache(B, Hq, H, 2)
    g = gu.GpuCache.__new__(gu.GpuCache)               # the helper class around an existing handle
    g.L, g.B, g.Hq, g.Hkv, g.max_ctx, g.G, g.ctx = L, B, Hq, H, n + 4, groups, ctx
    try:
        K = (rng.standard_normal((B, n, H, 64)) * 2).astype(np.float16)
        V = rng.standard_normal((B, n, H, 64)).astype(np.float16)
        bits = BITS[rng.choice(4, size=(B, n), p=[.4, .3, .2, .1])]
        g.append(1, K, V, bits)
        oc.append(K, V, bits)
        gu.assert_store_equals_oracle(g, 1, oc)
        for step in range(3):
            K = rng.standard_normal((B, 1, H, 64)).astype(np.float16)
            V = rng.standard_normal((B, 1, H, 64)).astype(np.float16)
            bits = BITS[rng.choice(4, size=(B, 1))]
            g.append(1, K, V, bits)
            oc.append(K, V, bits)
            Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
            gu.assert_attention_close(g.decode(1, Q), oc.decode_attn(Q), "step %d" % step)
    finally:
        g.close()
    torch.cuda.synchronize()
    lo, hi = buf[:guard].cpu().numpy(), buf[guard + need:].cpu().numpy()
    assert np.all(lo == 0xA5) and np.all(hi == 0xA5), "bytes outside the workspace were written"
    assert int(buf[guard:guard + 64].sum()) >= 0       # still the caller's memory after kvq_destroy
