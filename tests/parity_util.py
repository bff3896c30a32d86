"""Helpers of the GPU parity tests: error metric and small conveniences (no arithmetic of the method)."""
import numpy as np
import torch


def rel_err_rows(got, ref):
    """max_i |got_i - ref_i| / max(|ref_i|, rms(ref_row)), taken over all rows: the 'max relative error' of the
    parity bar, made robust to near-zero entries by flooring the denominator at the row's RMS."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    got = got.reshape(-1, got.shape[-1])
    ref = ref.reshape(-1, ref.shape[-1])
    if ref.size == 0:
        return 0.0
    rms = np.sqrt(np.mean(ref * ref, axis=-1, keepdims=True))
    den = np.maximum(np.abs(ref), np.maximum(rms, 1e-300))
    return float(np.max(np.abs(got - ref) / den))


def rel_err_stats(got, ref):
    """The same per-entry relative error as rel_err_rows, summarised three ways: its maximum, its root mean square
    and its 99.99th percentile over all entries."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    got = got.reshape(-1, got.shape[-1])
    ref = ref.reshape(-1, ref.shape[-1])
    if ref.size == 0:
        return dict(max=0.0, rms=0.0, p9999=0.0)
    rms = np.sqrt(np.mean(ref * ref, axis=-1, keepdims=True))
    e = np.abs(got - ref) / np.maximum(np.abs(ref), np.maximum(rms, 1e-300))
    return dict(max=float(e.max()), rms=float(np.sqrt(np.mean(e * e))), p9999=float(np.percentile(e, 99.99)))


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def to_dev(w, device="cuda"):
    out = {k: v.to(device) for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: v.to(device) for k, v in lw.items()} for lw in w["layers"]]
    return out


def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round float64 values to bf16 (round-to-nearest-even, as the GPU stores logits) and widen again."""
    return torch.from_numpy(np.asarray(a, np.float64)).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
