"""The allocation-free entry point, mmee_search_static, against the handle-based search.

Some embedders cannot let the library allocate device memory (their own pool owns the device, or a
cudaMalloc would stall a latency-critical loop), so this entry point keeps its scratch in a fixed
array inside the library.  That array is shared by all calls and keeps stale contents, which is
what this test exercises: two different searches back to back must each reproduce, byte for byte,
what mmee_create + mmee_search return for the same problem.  The result buffers are allocated here,
by the caller, before the calls.  Collected last on purpose.
"""
import pytest
import torch

import mmee_inputs as mi
import paper_2604_03446_b200.binding as mm

pytestmark = pytest.mark.gpu


def _handle_search(cfg, obj):
    best, topk = mm.result_buffer(1), mm.result_buffer(obj["topk"])
    h = mm.mmee_create(cfg["workload"], cfg["arch"], obj)
    try:
        mm.mmee_search(h, best, topk)
        torch.cuda.synchronize()
    finally:
        mm.mmee_destroy(h)
    return bytes(best.cpu().numpy().tobytes()), bytes(topk.cpu().numpy().tobytes())


def test_static_scratch_search_matches_the_handle_search_twice_in_a_row():
    first = mi.config1()
    obj1 = dict(first["searches"][0], topk=16)                       # energy, many feasible mappings
    second = mi.random_tiny_problem(5)
    obj2 = dict(second["searches"][0], objective=mi.OBJ_LATENCY, topk=3)    # other problem, other k
    cases = [(first, obj1), (second, obj2)]
    want = [_handle_search(cfg, obj) for cfg, obj in cases]

    bufs = [(mm.result_buffer(1), mm.result_buffer(obj["topk"])) for _, obj in cases]
    for (cfg, obj), (best, topk) in zip(cases, bufs):                # back to back, no sync between
        mm.mmee_search_static(cfg["workload"], cfg["arch"], obj, best, topk)
    torch.cuda.synchronize()
    for (best, topk), (want_best, want_topk) in zip(bufs, want):
        assert bytes(best.cpu().numpy().tobytes()) == want_best
        assert bytes(topk.cpu().numpy().tobytes()) == want_topk
    got = mm.read_results(bufs[0][0], 1)[0]
    assert got.status == mm.OK and got.n_total == 162067500 and got.idx != mm.NO_INDEX

    # What the entry point is for: once the first call on the device has looked the array up, further calls
    # take no device memory at all (the free-memory figure of the device does not move).
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        for (cfg, obj), (best, topk) in zip(cases, bufs):
            mm.mmee_search_static(cfg["workload"], cfg["arch"], obj, best, topk)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    for (best, topk), (want_best, want_topk) in zip(bufs, want):
        assert bytes(best.cpu().numpy().tobytes()) == want_best
        assert bytes(topk.cpu().numpy().tobytes()) == want_topk


def test_static_scratch_search_rejects_bad_arguments():
    cfg = mi.config1()
    best = mm.result_buffer(1)
    with pytest.raises(mm.MmeeError) as e:
        mm.mmee_search_static(cfg["workload"], cfg["arch"], dict(cfg["searches"][0], topk=17), best)
    assert e.value.code == mm.ERR_RANGE
    assert mm.library().mmee_search_static(None, None, None, None, None, None) == mm.ERR_ARG
