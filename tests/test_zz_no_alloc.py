"""netmax_read_columns_static: the sampled read-back for callers that cannot allocate.

A process that gave all of its device memory to a pool allocator (and therefore built its
context on a caller-owned workspace), a polling loop that cannot afford the device-wide
synchronisation of cudaMalloc / cudaFree, or code running where allocation is forbidden
cannot use netmax_read_columns, which allocates its staging buffers on every call.  The
static variant stages through a fixed array inside the library instead.  This test calls
it through the C ABI twice in a row (the second call finds the first call's data still in
the shared array) and requires exactly the values netmax_read_columns returns: both paths
copy fp32 values, so the comparison is bit for bit.  The file sorts last on purpose, so a
run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest

from paper_2009_05766_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nm():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2009_05766_b200 import binding
    binding.lib()
    return binding


def _policy(M, seed):
    P = np.random.default_rng(seed).random((M, M)) + 0.05
    np.fill_diagonal(P, 0.0)
    return P / P.sum(axis=1, keepdims=True)


def test_static_read_back_matches_allocating_read_back_twice_in_a_row(nm):
    M, d = 6, 50021
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=_policy(M, 1), sigma=0.1, x0_std=1.0, c_std=1.0, seed=31)
    g.round(4)
    first = workloads.sample_columns(d, 3000, 1)
    got1 = g.read_columns_static(first)
    assert got1.shape == (M, first.shape[0])
    assert (got1 == g.read_columns(first)).all()
    # second call, back to back: fewer and different columns, after the state has moved on;
    # whatever the first call left in the shared array must not leak into the result
    g.round(3)
    second = workloads.sample_columns(d, 700, 2)[::-1].copy()
    got2 = g.read_columns_static(second)
    assert (got2 == g.read_columns(second)).all()
    assert (got2 == g.read_replicas()[:, second]).all()
    assert not (got2[:, :50] == got1[:, :50]).all()
    g.close()


def test_static_read_back_is_shared_by_contexts_and_checks_its_limits(nm):
    M, d = 64, 9000
    a = nm.Netmax(M=M, d=d, lr=0.05, prob=_policy(M, 3), x0_std=1.0, c_std=1.0, seed=5)
    b = nm.Netmax(M=3, d=100, lr=0.05, prob=_policy(3, 4), x0_std=1.0, c_std=1.0, seed=6)
    cols = np.arange(0, 4096, dtype=np.int64)            # 64 * 4096 values: exactly the maximum
    assert (a.read_columns_static(cols) == a.read_columns(cols)).all()
    small = np.array([99, 0, 50], dtype=np.int64)
    assert (b.read_columns_static(small) == b.read_columns(small)).all()
    assert (a.read_columns_static(cols[:10]) == a.read_columns(cols[:10])).all()
    for ctx, bad in ((a, np.arange(0, 4097, dtype=np.int64)),       # too many values (and columns)
                     (b, np.zeros(4097, dtype=np.int64)),           # too many columns
                     (b, np.array([100], dtype=np.int64))):         # outside [0, d)
        with pytest.raises(nm.NetmaxError) as e:
            ctx.read_columns_static(bad)
        assert e.value.code == -1
    assert "staging area" in str(e.value) or "outside" in str(e.value)
    assert b.read_columns_static(np.zeros(0, dtype=np.int64)).shape == (3, 0)
    a.close()
    b.close()


def test_static_read_back_on_a_caller_owned_bfloat16_workspace_leaves_free_memory_alone(nm):
    """The case the entry point exists for: every device buffer of the context lives in memory the
    caller handed over (here a torch tensor, as a pool allocator would), the state is bfloat16 (the
    gather widens it), and across a call the device's free memory does not move."""
    import torch
    M, d, ring = 5, 30011, 64
    size = nm.Netmax.workspace_size(M, d, ring, storage="bf16")
    ws = torch.empty(size + 256, dtype=torch.uint8, device="cuda")
    ptr = (ws.data_ptr() + 255) // 256 * 256
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=_policy(M, 7), sigma=0.1, x0_std=1.0, c_std=1.0, seed=77, storage="bf16",
                  trace_rounds=ring, workspace=ptr, workspace_bytes=size)
    g.round(5)
    cols = workloads.sample_columns(d, 2000, 3)
    first = g.read_columns_static(cols)          # the first call on a device looks the array's address up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    second = g.read_columns_static(cols)
    third = g.read_columns_static(cols[::-1].copy())
    free_after = torch.cuda.mem_get_info()[0]
    assert free_after == free_before
    want = g.read_replicas()[:, cols]            # (a bfloat16 context stages this through its own spare buffer)
    assert (first == want).all() and (second == want).all() and (third == want[:, ::-1]).all()
    assert (want == nm_bf16_exact(want)).all()   # the values are bfloat16 codes, widened exactly
    g.close()
    del ws


def nm_bf16_exact(a):
    """fp32 values with the low 16 bits cleared: what an exactly widened bfloat16 looks like."""
    return (a.view(np.uint32) & np.uint32(0xFFFF0000)).view(np.float32)
