"""Helpers shared by the GPU parity tests: run the CUDA library and the CPU oracle on the same bytes."""
from __future__ import annotations

import numpy as np
import torch

import paper_2102_08124_b200 as tm
from oracle import tm_oracle as orc


def to_device(W: np.ndarray) -> torch.Tensor:
    """float32 array or uint16 bf16 patterns -> CUDA tensor of the same bytes."""
    if W.dtype == np.uint16:
        return torch.from_numpy(W.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(W).cuda()


def to_host_bits(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    if t.dtype == torch.float32:
        return t.view(torch.int32).cpu().numpy().view(np.uint32)
    return t.cpu().numpy().view(np.uint32)


def gpu_find_mask(W: np.ndarray, N, M, method, **kw):
    Wd = to_device(W)
    fn = tm.tm_find_mask_bf16 if W.dtype == np.uint16 else tm.tm_find_mask
    mask, masked, obj = fn(Wd, N, M, method, **kw)
    torch.cuda.synchronize()
    return dict(mask=to_host_bits(mask), masked=None if masked is None else to_host_bits(masked),
                objective=None if obj is None else float(obj.item()), status=tm.tm_device_status())


def oracle_bits(res, W):
    masked = res["masked"]
    if masked is not None:
        masked = masked.view(np.uint16) if W.dtype == np.uint16 else masked.view(np.uint32)
    return res["mask"], masked


def assert_parity(W: np.ndarray, N, M, method, threads=None, rel=1e-6):
    """Mask and masked weights bit-exact, objective within 1e-6 relative (fp32 sums on the GPU)."""
    want = orc.find_mask(W, N, M, method, threads=threads or orc.max_threads())
    got = gpu_find_mask(W, N, M, method)
    wm, wmasked = oracle_bits(want, W)
    assert np.array_equal(got["mask"], wm), "mask differs in %d words" % int((got["mask"] != wm).sum())
    assert np.array_equal(got["masked"], wmasked)
    if rel is not None:
        assert abs(got["objective"] - want["objective"]) <= rel * abs(want["objective"]) + 1e-300
    assert got["status"] == (tm.TM_DEV_NONFINITE if want["nonfinite"] else 0)
    return want, got
