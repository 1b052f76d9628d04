"""-m gpu: candidate-sharded selection (prism_select_sharded).

One GPU is all these tests get, so the ranks are THREADS of this process, each with its own handle and stream; the
score exchange is a host-side sum between the threads (stream synchronised on both sides), so no kernel ever
waits for another kernel.  What is checked is what has to hold on any number of GPUs: every rank returns exactly
what the unsharded call returns, bit for bit, for any partition of the candidates."""
import threading
from dataclasses import replace

import numpy as np
import pytest

import synth
from synth.configs import MODE_CLUSTER, MODE_NONE, Schedule

from test_gpu_select import MID, MID_WL, dev_i32, make_model, run

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_2510_15620_b200 as pkg
    return pkg


class HostSum:
    """Element-wise sum over `world` threads of a device vector, through the host."""

    def __init__(self, world):
        self.world, self.bar, self.parts, self.calls = world, threading.Barrier(world), [None] * world, 0

    def reducer(self, rank):
        def reduce(t):
            torch.cuda.current_stream().synchronize()
            self.parts[rank] = t.detach().cpu().numpy().copy()
            self.bar.wait(timeout=120)
            total = np.sum(np.stack([p[: t.numel()] for p in self.parts]), axis=0, dtype=np.float32)
            nz = np.sum(np.stack([p != 0 for p in self.parts]), axis=0)
            assert nz.max() <= 1                                   # one owner per candidate: the sum is exact
            self.bar.wait(timeout=120)                             # everyone has read before anyone overwrites
            t.copy_(torch.from_numpy(total).to(t.device))
            if rank == 0:
                self.calls += 1
        return reduce


def run_sharded(P, cfg, w, req, k, sched, owner, world, **model_kw):
    out, errs = [None] * world, []
    hs = HostSum(world)

    def work(rank):
        try:
            torch.cuda.set_device(0)
            with torch.cuda.stream(torch.cuda.Stream()):
                model = make_model(P, cfg, w, req, **model_kw)
                idx, sc, tr = model.select_sharded(dev_i32(req["query"]), dev_i32(req["cand_tokens"]),
                                                   dev_i32(req["cand_offsets"]), k, sched,
                                                   (owner == rank).astype(np.uint8), hs.reducer(rank))
                out[rank] = (idx.cpu().numpy(), sc.cpu().numpy(), tr)
                model.close()
        except BaseException as e:                                # noqa: BLE001 - reported by the main thread
            errs.append(e)
            hs.bar.abort()

    ts = [threading.Thread(target=work, args=(r,)) for r in range(world)]
    for t in ts:
        t.start()
    for t in ts:
        t.join(timeout=300)
    if errs:
        raise errs[0]
    assert all(o is not None for o in out)
    return out, hs.calls


@pytest.fixture(scope="module")
def mid_case(P):
    w = synth.make_weights(MID, seed=5)
    req = synth.make_request(MID_WL, 0)
    return w, req


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_equals_unsharded(P, mid_case, world):
    w, req = mid_case
    lens = np.diff(req["cand_offsets"]) + len(req["query"])
    owner = P.shard_candidates(lens, world)
    loads = np.array([lens[owner == r].sum() for r in range(world)])
    assert loads.max() - loads.min() <= lens.max()                 # greedy longest-first balances within one sequence
    base = make_model(P, MID, w, req)
    for sched in (MID_WL.schedule, replace(MID_WL.schedule, select_winners=0), Schedule(MODE_NONE)):
        ref_idx, ref_sc, ref_tr = run(P, base, req, MID_WL.top_k, sched)
        out, calls = run_sharded(P, MID, w, req, MID_WL.top_k, sched, owner, world)
        assert calls == len(ref_tr.records)                        # one exchange per scored layer, nothing else
        # the query's rows are shared on every rank too, and the ranks' token counts add up to the unsharded ones
        assert ref_tr.shared_prefix_rows == len(req["query"]) and all(o[2].shared_prefix_rows == len(req["query"]) for o in out)
        assert [sum(t) for t in zip(*[o[2].tokens_per_layer for o in out])] == ref_tr.tokens_per_layer
        assert [sum(r.tokens_before for r in recs) for recs in zip(*[o[2].records for o in out])] == \
               [r.tokens_before for r in ref_tr.records]
        for idx, sc, tr in out:
            assert np.array_equal(idx, ref_idx)
            assert np.array_equal(sc.view(np.uint32), ref_sc.view(np.uint32))
            assert len(tr.records) == len(ref_tr.records)
            for a, b in zip(tr.records, ref_tr.records):
                assert (a.layer, a.n_active_before, a.fired, a.n_selected, a.n_dropped, a.n_deferred, a.k_rem_after) == \
                       (b.layer, b.n_active_before, b.fired, b.n_selected, b.n_dropped, b.n_deferred, b.k_rem_after)
                assert a.active_ids == b.active_ids and a.cuts == b.cuts and a.cv == b.cv
                assert np.array_equal(np.asarray(a.scores).view(np.uint32), np.asarray(b.scores).view(np.uint32))
    base.close()


def test_sharded_with_an_idle_rank_and_a_single_owner(P, mid_case):
    """Degenerate partitions: one rank owns everything (the other runs no rows at all), and a rank that owns a
    single candidate which is dropped at the first probe and idles from then on."""
    w, req = mid_case
    n = MID_WL.n_candidates
    base = make_model(P, MID, w, req)
    ref_idx, ref_sc, ref_tr = run(P, base, req, MID_WL.top_k, MID_WL.schedule)
    dropped_first = [i for i in range(n) if i not in ref_tr.records[1].active_ids and i not in ref_idx][:1] if len(ref_tr.records) > 1 else []
    cases = [np.zeros(n, np.int32)]
    if dropped_first:
        o = np.zeros(n, np.int32)
        o[dropped_first[0]] = 1
        cases.append(o)
    for owner in cases:
        out, _ = run_sharded(P, MID, w, req, MID_WL.top_k, MID_WL.schedule, owner, 2)
        for idx, sc, _tr in out:
            assert np.array_equal(idx, ref_idx)
            assert np.array_equal(sc.view(np.uint32), ref_sc.view(np.uint32))
    base.close()


def test_sharded_fp32_path_and_chunked_streamed_models(P, mid_case):
    """The CUDA-core fp32 path (cfg 0) and a bf16 model that runs chunked under an activation budget with its
    layer weights streamed from pinned host memory: sharded over two ranks, both must return what the plain
    handle returns.  In the chunked case some chunks of a rank consist of other ranks' rowless sequences only."""
    wl = synth.workload(0)
    w0 = synth.make_weights(wl.model)
    r0 = synth.make_request(wl, 0)
    base = make_model(P, wl.model, w0, r0)
    ref = run(P, base, r0, wl.top_k, wl.schedule)
    owner = P.shard_candidates(np.diff(r0["cand_offsets"]) + len(r0["query"]), 2)
    for o in (owner, np.zeros_like(owner)):
        out, _ = run_sharded(P, wl.model, w0, r0, wl.top_k, wl.schedule, o, 2)
        for idx, sc, _tr in out:
            assert np.array_equal(idx, ref[0]) and np.array_equal(sc.view(np.uint32), ref[1].view(np.uint32))
    base.close()

    w, req = mid_case
    lens = np.diff(req["cand_offsets"]) + len(req["query"])
    per_tok = (1024 + 4096 + 2048 + 3072) * 2
    budget = 2 * int(lens.sum()) * 1024 * 4 + per_tok * (int(lens.max()) + 50)     # about one long sequence per chunk
    base = make_model(P, MID, w, req)
    ref = run(P, base, req, MID_WL.top_k, MID_WL.schedule)
    owner = (np.arange(MID_WL.n_candidates) >= MID_WL.n_candidates // 2).astype(np.int32)   # contiguous halves
    out, _ = run_sharded(P, MID, w, req, MID_WL.top_k, MID_WL.schedule, owner, 2,
                         activation_budget_bytes=budget, stream_weights=True)
    for idx, sc, tr in out:
        assert np.array_equal(idx, ref[0]) and np.array_equal(sc.view(np.uint32), ref[1].view(np.uint32))
        assert tr.n_chunks_max > 3
    base.close()


def test_sharded_argument_errors(P, mid_case):
    w, req = mid_case
    model = make_model(P, MID, w, req)
    with pytest.raises(ValueError):
        model.select_sharded(dev_i32(req["query"]), dev_i32(req["cand_tokens"]), dev_i32(req["cand_offsets"]), 4,
                             MID_WL.schedule, np.ones(3, np.uint8), lambda t: None)

    def boom(t):
        raise RuntimeError("exchange failed")

    with pytest.raises(RuntimeError, match="exchange failed"):
        model.select_sharded(dev_i32(req["query"]), dev_i32(req["cand_tokens"]), dev_i32(req["cand_offsets"]), 4,
                             MID_WL.schedule, np.ones(MID_WL.n_candidates, np.uint8), boom)
    # the handle is usable afterwards
    idx, sc, _ = model.select_sharded(dev_i32(req["query"]), dev_i32(req["cand_tokens"]), dev_i32(req["cand_offsets"]), 4,
                                      MID_WL.schedule, np.ones(MID_WL.n_candidates, np.uint8), lambda t: None)
    ref = run(P, model, req, 4, MID_WL.schedule)
    assert np.array_equal(idx.cpu().numpy(), ref[0])
    model.close()
