"""cvlc_decode_aggregate_noalloc: the aggregation entry point for callers that are not
allowed to allocate device memory (code living inside someone else's memory pool, plugins
barred from cudaMalloc after start-up, latency-critical loops).  It keeps its scratch in an
array built into the library, so the test checks that it gives what cvlc_decode_aggregate
gives, on two calls in a row that share that scratch, and that it refuses more clients than
the built-in scratch holds.  Collected last on purpose: a failure here stops nothing else."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _encode_clients(torch, B, n, d, seed0):
    dev = torch.device("cuda:0")
    streams = []
    for i in range(n):
        x = np.random.default_rng(seed0 + i).laplace(0, 1e-2, d).astype(np.float32)
        p = B.make_params(d, 10 * 4096, packet_bits=4096, seed=seed0 + i, client_id=i, scale_B=1.0 + 0.01 * i)
        enc = B.ClientEncoder(p, dev)
        out = enc.run(torch.from_numpy(x).to(dev))
        assert enc.status() == B.CVLC_OK
        streams.append(out.clone())
    return streams


def _tables(torch, streams, weights):
    dev = torch.device("cuda:0")
    ptrs = torch.tensor([s.data_ptr() for s in streams], dtype=torch.int64, device=dev)
    sizes = torch.tensor([s.numel() for s in streams], dtype=torch.int64, device=dev)
    w = torch.tensor(weights, dtype=torch.float32, device=dev)
    return ptrs, sizes, w


def _close(got, ref):
    got, ref = got.double().cpu().numpy(), ref.double().cpu().numpy()
    assert (np.abs(got - ref) <= 1e-7 + 1e-6 * np.abs(ref)).all()


def test_noalloc_matches_workspace_variant_on_two_calls_in_a_row():
    import torch
    from paper_2402_03770_b200 import binding as B
    assert torch.cuda.is_available()
    B.lib()
    B.cvlc_set_device(0)
    dev = torch.device("cuda:0")
    d = 50_000
    status = torch.full((1,), -1, dtype=torch.int32, device=dev)

    # call 1: seven clients, overwrite
    s1 = _encode_clients(torch, B, 7, d, seed0=10)
    p1, z1, w1 = _tables(torch, s1, [3, 1, 4, 1, 5, 9, 2])
    ref1 = torch.full((d,), float("nan"), dtype=torch.float32, device=dev)
    B.cvlc_decode_aggregate(p1, z1, w1, 7, 0.0, d, ref1, False, B.alloc_bytes(B.cvlc_decode_workspace_bytes(7), dev))
    got1 = torch.full((d,), float("nan"), dtype=torch.float32, device=dev)
    B.cvlc_decode_aggregate_noalloc(p1, z1, w1, 7, 0.0, d, got1, False, status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.CVLC_OK
    _close(got1, ref1)
    # ... and what the CPU oracle computes from the same streams
    import oracle as O
    want1 = O.decode_aggregate([s.cpu().numpy() for s in s1], np.array([3, 1, 4, 1, 5, 9, 2], np.float32), d)
    _close(got1, torch.from_numpy(want1))

    # call 2, right after, fewer clients and accumulating: nothing of call 1 may leak through the scratch
    s2 = _encode_clients(torch, B, 3, d, seed0=40)
    p2, z2, w2 = _tables(torch, s2, [2, 2, 6])
    base = torch.linspace(-1, 1, d, dtype=torch.float32, device=dev)
    ref2 = base.clone()
    B.cvlc_decode_aggregate(p2, z2, w2, 3, 25.0, d, ref2, True, B.alloc_bytes(B.cvlc_decode_workspace_bytes(3), dev))
    got2 = base.clone()
    status.fill_(-1)
    B.cvlc_decode_aggregate_noalloc(p2, z2, w2, 3, 25.0, d, got2, True, status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.CVLC_OK
    _close(got2, ref2)

    # a malformed stream is reported through the caller's status word, and the next call is clean again
    bad = s2[1].clone()
    bad[0] = 0
    p3, z3, w3 = _tables(torch, [s2[0], bad, s2[2]], [1, 1, 1])
    B.cvlc_decode_aggregate_noalloc(p3, z3, w3, 3, 0.0, d, got2, False, status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.CVLC_ERR_BAD_STREAM
    B.cvlc_decode_aggregate_noalloc(p1, z1, w1, 7, 0.0, d, got1, False, status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.CVLC_OK
    _close(got1, ref1)


def test_noalloc_at_its_largest_client_count():
    """exactly NOALLOC_MAX_CLIENTS small streams: the built-in scratch is used to its last table entry"""
    import torch
    import oracle as O
    from paper_2402_03770_b200 import binding as B
    B.lib()
    B.cvlc_set_device(0)
    dev = torch.device("cuda:0")
    d, n = 3000, B.NOALLOC_MAX_CLIENTS
    host_streams = []
    for i in range(n):
        x = np.random.default_rng(900 + i).standard_normal(d).astype(np.float32)
        po = O.make_params(d, 2 * 1024, packet_bits=1024, seed=i, client_id=i)
        host_streams.append(O.encode(x, po, O.plan(x, po)))
    weights = np.random.default_rng(5).uniform(1, 9, n).astype(np.float32)
    streams = [torch.from_numpy(s).to(dev) for s in host_streams]
    ptrs, sizes, w = _tables(torch, streams, weights.tolist())
    status = torch.full((1,), -1, dtype=torch.int32, device=dev)
    got = torch.full((d,), float("nan"), dtype=torch.float32, device=dev)
    B.cvlc_decode_aggregate_noalloc(ptrs, sizes, w, n, 0.0, d, got, False, status)
    ref = torch.full((d,), float("nan"), dtype=torch.float32, device=dev)
    B.cvlc_decode_aggregate(ptrs, sizes, w, n, 0.0, d, ref, False, B.alloc_bytes(B.cvlc_decode_workspace_bytes(n), dev))
    torch.cuda.synchronize()
    assert int(status.item()) == B.CVLC_OK
    _close(got, ref)
    _close(got, torch.from_numpy(O.decode_aggregate(host_streams, weights, d)))


def test_noalloc_rejects_more_clients_than_its_scratch_holds():
    import torch
    from paper_2402_03770_b200 import binding as B
    B.lib()
    B.cvlc_set_device(0)
    dev = torch.device("cuda:0")
    n = B.NOALLOC_MAX_CLIENTS + 1
    z = torch.zeros(n, dtype=torch.int64, device=dev)
    w = torch.ones(n, dtype=torch.float32, device=dev)
    out = torch.zeros(1000, dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(B.CvlcError) as e:
        B.cvlc_decode_aggregate_noalloc(z, z, w, n, 0.0, 1000, out, False, status)
    assert e.value.code == B.CVLC_ERR_WORKSPACE_TOO_SMALL
