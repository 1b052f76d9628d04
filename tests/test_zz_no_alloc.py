"""-m gpu: prism_op_route_static, the pruning decision for callers that cannot allocate device memory
(a host whose own pool already owns the GPU, or a loop that must not stall on cudaMalloc/cudaFree),
must give exactly what prism_op_route gives.  Collected last on purpose; passes alone and after the
other tests."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

MODE_CLUSTER = 2


def _buffers(n, n_result):
    return dict(cu_new=torch.full((n + 1,), -7, dtype=torch.int32, device="cuda"),
                s2o_new=torch.full((n,), -7, dtype=torch.int32, device="cuda"),
                oon=torch.full((n,), -7, dtype=torch.int32, device="cuda"),
                ridx=torch.full((n + n_result,), -7, dtype=torch.int32, device="cuda"),
                rsc=torch.zeros(n + n_result, dtype=torch.float32, device="cuda"))


def _call(fn, P, scores, cu, ids, n, k_rem, n_result, n_clusters, thr):
    b = _buffers(n, n_result)
    state = torch.tensor([n, int(cu[-1]), k_rem, n_result, 0, 0, 0, 0], dtype=torch.int32, device="cuda")
    rec = torch.zeros(P.ops.RECORD_BYTES, dtype=torch.uint8, device="cuda")
    fn(scores, cu, ids, n, MODE_CLUSTER, 0, thr, n_clusters, 0, 1, 0, 5, b["cu_new"], b["s2o_new"], b["oon"], state,
       b["ridx"], b["rsc"], rec)
    torch.cuda.synchronize()
    out = {k: v.cpu().numpy() for k, v in b.items()}
    out["state"] = state.cpu().numpy()
    out["rec"] = rec.cpu().numpy()
    return out


def test_route_static_equals_route_on_two_calls_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2510_15620_b200 as P
    rng = np.random.default_rng(2024)
    # two different problems back to back: the second call finds the first call's leftovers in the
    # shared scratch and must not be affected by them (the larger problem goes first)
    for n, k_rem, n_clusters, thr in ((1000, 20, 3, 0.2), (137, 9, 5, 0.0)):
        sc = (rng.normal(size=n) * 2 + 0.5).astype(np.float32)
        sc[rng.integers(0, n, size=n // 4)] = sc[1]                       # ties at the cuts
        lens = rng.integers(1, 300, size=n)
        cu = np.zeros(n + 1, np.int32)
        cu[1:] = np.cumsum(lens)
        scores = torch.from_numpy(sc).cuda()
        cu_d = torch.from_numpy(cu).cuda()
        ids = torch.arange(n, dtype=torch.int32, device="cuda")
        ref = _call(P.ops.prism_op_route, P, scores, cu_d, ids, n, k_rem, 3, n_clusters, thr)
        got = _call(P.ops.prism_op_route_static, P, scores, cu_d, ids, n, k_rem, 3, n_clusters, thr)
        assert int(ref["state"][0]) < n                                  # the case really prunes
        for key in ref:                                                    # integer and float outputs: bit for bit
            assert np.array_equal(ref[key], got[key]), key


def test_route_static_rejects_sizes_beyond_its_scratch():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2510_15620_b200 as P
    n = 1025
    z = torch.zeros(n + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(P.PrismError) as e:
        P.ops.prism_op_route_static(torch.zeros(n, device="cuda"), z, z, n, MODE_CLUSTER, 0, 0.0, 3, 0, 1, 0, 1, z, z, z,
                                    torch.zeros(8, dtype=torch.int32, device="cuda"), z, torch.zeros(n, device="cuda"), None)
    assert e.value.status == -2
