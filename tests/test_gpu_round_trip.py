"""netmax_round_from_host: one call that uploads replicas and centres, runs rounds and downloads the
result, pipelined over column chunks.  It must equal set_replicas + set_centres + round +
read_replicas bit for bit (replicas, peer trace, round counter) and in telemetry up to the order
of the chunk sums."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nm():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2009_05766_b200 import binding
    binding.lib()
    return binding


def random_policy(M, rng):
    P = rng.random((M, M)) + 0.05
    np.fill_diagonal(P, 0.0)
    return P / P.sum(axis=1, keepdims=True)


# (M, d, fuse_rounds, storage, chunks): fused tiles, one launch per round, cluster-resident tiles, a ragged
# tail, a chunk count that does not divide the vector, and the shapes that fall back to the plain sequence
CASES = [(8, 400_003, 0, "f32", 0), (8, 400_003, 1, "f32", 5), (3, 310_001, 0, "f32", 32), (64, 90_002, 0, "f32", 3),
         (16, 330_000, 3, "f32", 7), (5, 4_099, 0, "f32", 4), (8, 700_003, 0, "bf16", 4)]


@pytest.mark.parametrize("M,d,fuse,storage,chunks", CASES)
def test_round_trip_equals_the_four_calls(nm, M, d, fuse, storage, chunks):
    rng = np.random.default_rng(M + d)
    P = random_policy(M, rng)
    kw = dict(M=M, d=d, lr=0.05, prob=P, sigma=0.1, objective=1, seed=3, trace_rounds=16, fuse_rounds=fuse, storage=storage)
    x = rng.standard_normal((M, d)).astype(np.float32)
    c = rng.standard_normal((M, d)).astype(np.float32)
    a, b = nm.Netmax(**kw), nm.Netmax(**kw)
    out = np.empty((M, d), dtype=np.float32)
    for step, n in enumerate((5, 1, 7)):
        a.set_replicas(x)
        a.set_centres(c)
        a.round(n)
        want = a.read_replicas()
        b.round_from_host(x, c, n, out, chunks)
        assert (out.view(np.uint32) == want.view(np.uint32)).all(), step
        assert b.rounds_done == a.rounds_done
        assert (b.peer_trace(a.rounds_done - n, n) == a.peer_trace(a.rounds_done - n, n)).all()
        (ca, la), (cb, lb) = a.telemetry(a.rounds_done - n, n), b.telemetry(b.rounds_done - n, n)
        np.testing.assert_allclose(cb, ca, rtol=1e-6)
        np.testing.assert_allclose(lb, la, rtol=1e-6)
        x = want + np.float32(0.25)           # the next step starts from new host data
    # without new inputs the call continues from the state on the device, as round + read do
    a.round(3)
    b.round_from_host(None, None, 3, out, chunks)
    assert (out.view(np.uint32) == a.read_replicas().view(np.uint32)).all()
    # and the context is left as the four calls leave it
    a.round(2)
    b.round(2)
    assert (a.read_replicas().view(np.uint32) == b.read_replicas().view(np.uint32)).all()
    a.close()
    b.close()


def test_round_trip_through_pinned_buffers_and_its_argument_checks(nm):
    import torch
    M, d = 4, 500_001
    P = random_policy(M, np.random.default_rng(2))
    stream = torch.cuda.Stream()
    g = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.05, seed=9, trace_rounds=8, stream=stream.cuda_stream)
    h = nm.Netmax(M=M, d=d, lr=0.05, prob=P, sigma=0.05, seed=9, trace_rounds=8)
    hx = torch.randn((M, d), dtype=torch.float32).pin_memory()
    hc = torch.randn((M, d), dtype=torch.float32).pin_memory()
    ho = torch.empty((M, d), dtype=torch.float32).pin_memory()
    g.round_from_host(hx.data_ptr(), hc.data_ptr(), 4, ho.data_ptr(), 6)
    h.set_replicas(hx.numpy())
    h.set_centres(hc.numpy())
    h.round(4)
    assert (ho.numpy().view(np.uint32) == h.read_replicas().view(np.uint32)).all()
    out = np.empty((M, d), dtype=np.float32)
    g.round_from_host(None, None, 20, out, 6)        # more rounds than the trace ring holds: the plain sequence
    h.round(20)
    assert (out.view(np.uint32) == h.read_replicas().view(np.uint32)).all()
    for bad in (dict(n_rounds=-1, n_chunks=0), dict(n_rounds=1, n_chunks=33), dict(n_rounds=1, n_chunks=-1)):
        with pytest.raises(nm.NetmaxError) as e:
            g.round_from_host(None, None, bad["n_rounds"], out, bad["n_chunks"])
        assert e.value.code == -1
    assert nm.lib().netmax_round_from_host(g._h, None, None, 1, None, 0) == -1
    g.close()
    h.close()
