"""The allocation-free entry point.  Some callers (a plug-in living inside another framework's memory
pool, a loop that pre-allocates everything) cannot call cudaMalloc or hand the library a workspace sized
up front; tm_find_mask_batched_static() serves them from a scratch array built into the library.  This
test calls it through the C ABI twice in a row and demands the results of tm_find_mask_batched().
Collected last on purpose, so that a run stopping at the first failure has already run everything else."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_2102_08124_b200 as tm
import workloads
from oracle import tm_oracle as orc
from paper_2102_08124_b200 import binding

pytestmark = pytest.mark.gpu


def _host_matrices(M):
    # 132 bf16 columns give a row pitch that is not a multiple of 16 bytes (the generic kernel takes it);
    # the 4:8 search needs multiples of 8
    return [workloads.normal_f32(64, 520, 0.02, 901), workloads.quantised_bf16(128, 1024, 0.02, 902),
            workloads.normal_bf16(16, 132 if M == 4 else 136, 0.02, 903), workloads.normal_f32(8, 8, 1.0, 904)]


def _device_tensors(M):
    mats = _host_matrices(M)
    out = []
    for m in mats:
        if m.dtype == np.uint16:
            out.append(torch.from_numpy(m.view(np.int16)).cuda().view(torch.bfloat16))
        else:
            out.append(torch.from_numpy(m).cuda())
    return out


def _bits(t):
    return t.view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32).cpu().numpy()


@pytest.mark.parametrize("N,M,method", [(2, 4, tm.TM_APPROX), (2, 4, tm.TM_EXACT), (4, 8, tm.TM_APPROX)])
def test_static_scratch_entry_matches_the_workspace_entry(N, M, method):
    Ws = _device_tensors(M)
    ref_masks, ref_maskeds, ref_obj, ref_status, _ = tm.tm_find_mask_batched(Ws, N, M, method)
    torch.cuda.synchronize()
    # everything the call writes is allocated here, by the test; the call itself allocates nothing
    masks = [torch.empty_like(m) for m in ref_masks]
    maskeds = [torch.empty_like(w) for w in Ws]
    obj = torch.empty_like(ref_obj)
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    for round_ in range(2):                                     # two calls in a row share the built-in scratch
        for t in masks + maskeds:
            t.view(torch.uint8).fill_(0xA5)
        obj.fill_(-1.0)
        tm.tm_find_mask_batched_static(Ws, N, M, method, masks, maskeds, obj, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for k in range(len(Ws)):
            assert np.array_equal(masks[k].cpu().numpy(), ref_masks[k].cpu().numpy()), (round_, k)
            assert np.array_equal(_bits(maskeds[k]), _bits(ref_maskeds[k])), (round_, k)
        assert np.array_equal(obj.cpu().numpy(), ref_obj.cpu().numpy()), round_   # same kernels, same order: same bits
    # and, directly, the CPU oracle's answer on the same bytes
    oracle_method = {tm.TM_APPROX: orc.APPROX, tm.TM_EXACT: orc.EXACT}[method]
    for k, m in enumerate(_host_matrices(M)):
        want = orc.find_mask(m, N, M, oracle_method)
        assert np.array_equal(masks[k].cpu().numpy().view(np.uint32), want["mask"]), k
        assert np.array_equal(_bits(maskeds[k]).view(np.uint16 if m.dtype == np.uint16 else np.uint32),
                              want["masked"].view(np.uint16 if m.dtype == np.uint16 else np.uint32)), k
        assert abs(float(obj[k].item()) - want["objective"]) <= 1e-6 * abs(want["objective"])


def test_static_scratch_entry_rejects_too_many_matrices():
    lib = tm.load_library()
    n = tm.TM_STATIC_MAX_MATRICES + 1
    W = torch.zeros((4, 4), device="cuda")
    mask = torch.zeros((4, 1), dtype=torch.int32, device="cuda")
    arr = (binding.tm_problem * n)()
    for k in range(n):
        arr[k].W = W.data_ptr(); arr[k].rows = 4; arr[k].cols = 4; arr[k].ld = 4; arr[k].dtype = 0
        arr[k].mask_out = mask.data_ptr(); arr[k].masked_w_out = None; arr[k].objective_out = None
    rc = lib.tm_find_mask_batched_static(arr, n, 2, 4, tm.TM_APPROX, None, None)
    assert rc == 9 and "too many" in tm.tm_status_string(rc)
    assert lib.tm_find_mask_batched_static(arr, tm.TM_STATIC_MAX_MATRICES, 2, 4, tm.TM_APPROX, None, None) == 0
    torch.cuda.synchronize()
    assert lib.tm_find_mask_batched_static(None, 0, 2, 4, tm.TM_APPROX, None, None) == 0
