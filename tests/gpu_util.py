"""Helpers shared by the GPU parity tests: tensors onto the device, error metrics, routing checks."""
import numpy as np
import torch

GAP = 1e-3          # selections must match the oracle exactly where the k-th/(k+1)-th logit gap exceeds this


def torch_dtype(name):
    return torch.float32 if name == "f32" else torch.bfloat16


def to_dev(w, *names):
    """Workload tensors as CUDA tensors of the workload's storage type (bf16 values convert exactly)."""
    dt = torch_dtype(w.dtype)
    return [torch.from_numpy(np.ascontiguousarray(w[n])).to("cuda").to(dt) for n in names]


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def max_abs(a, b):
    return float(np.max(np.abs(np.asarray(a, np.float64) - np.asarray(b, np.float64)))) if np.size(a) else 0.0


def bf16_bound_ok(y, ref):
    """Per-element bound of a bf16 result against the fp64 oracle: 5e-2 absolute plus one bf16 ulp of the
    reference (2^-8 |ref|, twice the half-ulp the single rounding of y may cost).  Returns the worst excess."""
    y = np.asarray(y, np.float64)
    ref = np.asarray(ref, np.float64)
    if not y.size:
        return 0.0
    return float(np.max(np.abs(y - ref) - (5e-2 + 2.0 ** -8 * np.abs(ref))))


def clear_tokens(oracle_logits, k):
    """Tokens whose selection is fixed: the k-th / (k+1)-th logit gap and the gaps between consecutive picks exceed GAP."""
    lg = np.asarray(oracle_logits, np.float64)
    N = lg.shape[1]
    srt = -np.sort(-lg, axis=1)
    gap = srt[:, k - 1] - srt[:, k] if k < N else np.full(lg.shape[0], np.inf)
    inner = np.min(srt[:, :k - 1] - srt[:, 1:k], axis=1) if k > 1 else np.full(lg.shape[0], np.inf)
    return (gap > GAP) & (inner > GAP)


def check_selection(gpu_idx, oracle_idx, oracle_logits, k):
    """Exact match where the logit gap is clear; inside the band the GPU's set must still be a valid top-k."""
    gpu_idx = np.asarray(gpu_idx)
    lg = np.asarray(oracle_logits, np.float64)
    N = lg.shape[1]
    srt = -np.sort(-lg, axis=1)
    gap = srt[:, k - 1] - srt[:, k] if k < N else np.full(lg.shape[0], np.inf)
    # also the order of the picks is only fixed where consecutive selected logits are clearly apart
    inner = np.min(srt[:, :k - 1] - srt[:, 1:k], axis=1) if k > 1 else np.full(lg.shape[0], np.inf)
    clear = (gap > GAP) & (inner > GAP)
    np.testing.assert_array_equal(gpu_idx[clear], np.asarray(oracle_idx)[clear])
    for t in np.nonzero(~clear)[0]:
        chosen = gpu_idx[t]
        assert len(set(chosen.tolist())) == k and chosen.min() >= 0 and chosen.max() < N
        rest = np.delete(lg[t], chosen)
        if rest.size:
            assert lg[t, chosen].min() >= rest.max() - GAP
        assert np.all(np.diff(lg[t, chosen]) <= GAP)
    return clear
