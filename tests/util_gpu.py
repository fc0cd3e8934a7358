"""Helpers shared by the GPU parity tests: moving seeded host inputs to the device and the error
measures the tolerances are stated in."""
import numpy as np
import torch


def dev(a, dtype=None):
    """Host numpy -> CUDA tensor.  dtype 'bf16' narrows values that already sit on the bf16 grid."""
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    if dtype == "bf16":
        t = t.to(torch.bfloat16)
    return t.contiguous()


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64) if t.is_floating_point() else t.detach().cpu().numpy()


def max_rel_err(got, ref):
    """max |got - ref| / max |ref| over the tensor (the layer-output measure)."""
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    return float(np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-300))


def score_rel_err(got, ref):
    """max elementwise |got - ref| / ref (scores are positive)."""
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    return float((np.abs(got - ref) / np.maximum(np.abs(ref), 1e-300)).max())


def assert_kept_matches(kept_gpu, kept_ref, scores_ref, tol=1e-4):
    """Kept sets must be identical except for swaps among tokens whose oracle scores lie within
    `tol` (relative) of the selection threshold; the GPU list must be strictly ascending."""
    kept_gpu = np.asarray(kept_gpu).astype(np.int64)
    kept_ref = np.asarray(kept_ref).astype(np.int64)
    assert kept_gpu.shape == kept_ref.shape
    if len(kept_gpu) == 0:
        return 0
    assert np.all(np.diff(kept_gpu) > 0), "kept indices not strictly ascending"
    assert kept_gpu.min() >= 0 and kept_gpu.max() < len(scores_ref)
    only_gpu = np.setdiff1d(kept_gpu, kept_ref)
    only_ref = np.setdiff1d(kept_ref, kept_gpu)
    assert len(only_gpu) == len(only_ref)
    if len(only_gpu):
        thr = np.min(np.asarray(scores_ref)[kept_ref])
        for i in np.concatenate([only_gpu, only_ref]):
            assert abs(scores_ref[i] - thr) <= tol * abs(thr), (i, scores_ref[i], thr)
    return len(only_gpu)
