"""The refresh loop of sparse training from scratch: prepared plans, CUDA-graph replay, changed-bit counts (GPU),
and the straight-through masked layer (CPU)."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_2102_08124_b200 as tm
import workloads
from oracle import tm_oracle as orc
from paper_2102_08124_b200.refresh import MaskRefresher, masked_linear
from tests.gpu_util import to_device, to_host_bits


def test_masked_linear_straight_through_on_cpu():
    torch.manual_seed(0)
    W = torch.randn(8, 16, dtype=torch.float64, requires_grad=True)
    S = torch.from_numpy(orc.unpack_mask(orc.find_mask(W.detach().float().numpy(), 2, 4, orc.APPROX)["mask"], 16).astype(np.float64))
    x = torch.randn(5, 16, dtype=torch.float64, requires_grad=True)
    y = masked_linear(x, W, (W * S).detach())
    gy = torch.randn_like(y)
    y.backward(gy)
    assert torch.allclose(y, x @ (W * S).t())
    assert torch.allclose(x.grad, gy @ (W * S).detach())          # backward product uses the same (transposable) mask
    assert torch.allclose(W.grad, gy.t() @ x.detach())            # dense copy receives the unmasked gradient
    bits = S.numpy().reshape(2, 4, 4, 4)
    assert (bits.sum(axis=1) == 2).all() and (bits.sum(axis=3) == 2).all()   # so W*S and (W*S)^T are both 2:4


@pytest.mark.gpu
@pytest.mark.parametrize("N,M,method", [(2, 4, tm.TM_APPROX), (4, 8, tm.TM_APPROX), (2, 4, tm.TM_EXACT)])
def test_plan_equals_batched_call(N, M, method):
    mats = [workloads.normal_f32(32, 264, 0.05, 81), workloads.normal_bf16(64, 520, 0.02, 82), workloads.normal_bf16(16, 136, 0.02, 83)]
    Ws = [to_device(m) for m in mats]
    ref_masks, ref_maskeds, ref_obj, _, _ = tm.tm_find_mask_batched(Ws, N, M, method)
    plan = tm.tm_plan_create(Ws, N, M, method)
    for _ in range(2):
        masks, maskeds, objs, status = tm.tm_plan_run(plan)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for k in range(len(Ws)):
            assert np.array_equal(to_host_bits(masks[k]), to_host_bits(ref_masks[k]))
            assert np.array_equal(to_host_bits(maskeds[k]), to_host_bits(ref_maskeds[k]))
        # a plan's launch adds up its own partial sums, in another fixed order than the batched call's reduction kernel
        assert np.allclose(objs.cpu().numpy(), ref_obj.cpu().numpy(), rtol=1e-12, atol=0.0)
    # and, directly, the CPU oracle's answer on the same bytes
    for k, m in enumerate(mats):
        want = orc.find_mask(m, N, M, {tm.TM_APPROX: orc.APPROX, tm.TM_EXACT: orc.EXACT}[method])
        assert np.array_equal(to_host_bits(masks[k]), want["mask"])
        assert np.array_equal(to_host_bits(maskeds[k]), want["masked"].view(np.uint16 if m.dtype == np.uint16 else np.uint32))
        assert abs(float(objs[k].item()) - want["objective"]) <= 1e-6 * abs(want["objective"])
    tm.tm_plan_destroy(plan)


@pytest.mark.gpu
@pytest.mark.parametrize("N,M,method", [(2, 4, tm.TM_APPROX), (4, 8, tm.TM_APPROX), (2, 4, tm.TM_EXACT), (2, 4, tm.TM_APPROX_COVER)])
def test_plan_reduces_its_own_objectives(N, M, method):
    """Many matrices of one dtype in a plan: one launch whose last thread block adds up every matrix's partial sums.  Sizes from
    a single work item (most warps idle) to thousands (every warp holds several matrices or a piece of one), an empty matrix in
    the middle; run three times in a row (the count of finished blocks must return to zero)."""
    shapes = [(8, 520), (256, 2056), (8, 8), (0, 64), (1024, 4096), (16, 136), (64, 1032), (8, 16), (2048, 1024), (40, 3080)]
    mats = [workloads.quantised_bf16(r, c, 0.02, 300 + i) if r else np.zeros((0, c), np.uint16) for i, (r, c) in enumerate(shapes)]
    Ws = [to_device(m) if m.size else torch.empty((0, m.shape[1]), dtype=torch.bfloat16, device="cuda") for m in mats]
    plan = tm.tm_plan_create(Ws, N, M, method)
    omethod = {tm.TM_APPROX: orc.APPROX, tm.TM_EXACT: orc.EXACT, tm.TM_APPROX_COVER: orc.APPROX_COVER}[method]
    want = [orc.find_mask(m, N, M, omethod) if m.size else None for m in mats]
    for rep in range(3):
        plan.batch.objectives.fill_(-1.0)
        masks, maskeds, objs, status = tm.tm_plan_run(plan)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for k, m in enumerate(mats):
            if want[k] is None:
                assert float(objs[k].item()) == 0.0
                continue
            assert np.array_equal(to_host_bits(masks[k]), want[k]["mask"]), (rep, k)
            assert np.array_equal(to_host_bits(maskeds[k]), want[k]["masked"].view(np.uint16)), (rep, k)
            assert abs(float(objs[k].item()) - want[k]["objective"]) <= 1e-6 * abs(want[k]["objective"]), (rep, k)
    tm.tm_plan_destroy(plan)


@pytest.mark.gpu
def test_multi_matrix_call_is_refused_on_a_capturing_stream():
    """A call that must copy descriptor tables from host memory cannot be recorded: it returns TM_ERR_CAPTURE and
    enqueues nothing; the prepared plan on the same buffers can be recorded and replayed."""
    mats = [workloads.normal_bf16(16, 520, 0.02, 84), workloads.normal_bf16(16, 264, 0.02, 85)]
    Ws = [to_device(m) for m in mats]
    batch = tm.TmBatch(Ws)
    batch.run(2, 4, tm.TM_APPROX)                                   # outside a capture: fine
    plan = tm.tm_plan_create(Ws, 2, 4, tm.TM_APPROX)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    refused = None
    with torch.cuda.graph(graph, stream=side):
        try:
            batch.run(2, 4, tm.TM_APPROX, stream=side)
        except tm.TmError as e:
            refused = e.code
        tm.tm_plan_run(plan, stream=side)
    assert refused == 10 and "captured" in tm.tm_status_string(10)
    for t in plan.batch.masks:
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    for k, m in enumerate(mats):
        assert np.array_equal(to_host_bits(plan.batch.masks[k]), orc.find_mask(m, 2, 4, orc.APPROX, want_masked=False)["mask"])
    tm.tm_plan_destroy(plan)


@pytest.mark.gpu
def test_mask_hamming():
    rng = np.random.Generator(np.random.PCG64(91))
    for n in (1, 33, 4096, 100003):
        a = rng.integers(0, 2 ** 32, size=n, dtype=np.uint64).astype(np.uint32); b = rng.integers(0, 2 ** 32, size=n, dtype=np.uint64).astype(np.uint32)
        want = int(np.unpackbits((a ^ b).view(np.uint8)).sum())
        got = tm.tm_mask_hamming(torch.from_numpy(a.view(np.int32)).cuda(), torch.from_numpy(b.view(np.int32)).cuda())
        assert int(got.item()) == want
        if n > 40:                                                   # masks that start off a 16-byte boundary
            ad, bd = torch.from_numpy(a.view(np.int32)).cuda()[1:], torch.from_numpy(b.view(np.int32)).cuda()[3:n - 2 + 3 - 1]
            m = min(ad.numel(), bd.numel())
            got = tm.tm_mask_hamming(ad[:m], bd[:m])
            assert int(got.item()) == int(np.unpackbits((a[1:1 + m] ^ b[3:3 + m]).view(np.uint8)).sum())


@pytest.mark.gpu
@pytest.mark.parametrize("use_graph", [False, True])
def test_refresh_loop(use_graph):
    mats = workloads.config3(layers=1)                               # four BERT-large-shaped bf16 matrices
    Ws = [to_device(m) for m in mats]
    r = MaskRefresher(Ws, N=4, M=8, period=40, use_graph=use_graph)
    for k, m in enumerate(mats):
        assert np.array_equal(to_host_bits(r.masks[k]), orc.find_mask(m, 4, 8, orc.APPROX, threads=orc.max_threads(), want_masked=False)["mask"])
    assert r.refresh() == 0                                           # unchanged weights: no bit flips
    # a simulated optimizer update on the dense copies, then iterations 1..80: refreshes at 40 and 80
    mats2 = workloads.config3_perturbed(mats, 1)
    for W, m in zip(Ws, mats2):
        W.copy_(to_device(m))
    did = [it for it in range(1, 81) if r.step(it)]
    assert did == [40, 80]
    torch.cuda.synchronize()
    want = [orc.find_mask(m, 4, 8, orc.APPROX, threads=orc.max_threads()) for m in mats2]
    old = [orc.find_mask(m, 4, 8, orc.APPROX, threads=orc.max_threads(), want_masked=False)["mask"] for m in mats]
    flips = 0
    for k in range(len(mats)):
        assert np.array_equal(to_host_bits(r.masks[k]), want[k]["mask"])
        assert np.array_equal(to_host_bits(r.masked_weights[k]), want[k]["masked"])
        flips += int(np.unpackbits((want[k]["mask"] ^ old[k]).view(np.uint8)).sum())
    assert r.changed_bits[-2:] == [flips, 0] and flips > 0
