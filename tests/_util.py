"""Helpers shared by the GPU parity tests (no arithmetic of the method lives here)."""
import numpy as np
import torch


def bf16_to_torch(bits: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def torch_bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def to_dev(a: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def compare_accept(gpu_len, gpu_tok, ora, K, tol=1e-5):
    """Bit-exact comparison of accepted lengths and tokens with the stated exemptions.

    A sequence is exempt from the first position whose acceptance decision lies within `tol` of the
    threshold (|u - min(1, p/q)| < tol), and its token is exempt when the resample draw lies within
    `tol` (as a fraction of the residual mass) of a CDF boundary.  Returns counts.
    """
    gpu_len = np.asarray(gpu_len); gpu_tok = np.asarray(gpu_tok)
    B = len(gpu_len)
    n_exempt_accept = n_exempt_resample = n_checked = 0
    bad = []
    for b in range(B):
        olen = int(ora["accept_len"][b])
        examined = min(olen + 1, K)
        margins = ora["accept_margin"][b, :examined]
        if (margins < tol).any():
            n_exempt_accept += 1
            continue
        if gpu_len[b] != olen:
            bad.append((b, "len", int(gpu_len[b]), olen))
            continue
        if ora["resample_margin"][b] < tol:
            n_exempt_resample += 1
            continue
        n_checked += 1
        if gpu_tok[b] != ora["token"][b]:
            bad.append((b, "tok", int(gpu_tok[b]), int(ora["token"][b])))
    return dict(bad=bad, exempt_accept=n_exempt_accept, exempt_resample=n_exempt_resample, checked=n_checked)
