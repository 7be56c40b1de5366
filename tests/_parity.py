"""Helpers for the GPU-vs-oracle parity tests: run both sides on the same bytes and compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import tsq_ref as R
from paper_2511_04002_b200 import binding as B
from paper_2511_04002_b200 import synth


def dt_code(x: torch.Tensor) -> int:
    return R.F16 if x.dtype == torch.float16 else R.BF16


def gpu_encode(plan: B.Plan, x_cpu: torch.Tensor, ws=None, blob=None):
    """Encode on the GPU through the C ABI; returns (blob on device, host copy as uint8 numpy, ws)."""
    T = x_cpu.shape[0]
    if blob is None or ws is None:
        blob, ws = plan.alloc(T)
    x = x_cpu.cuda()
    plan.encode(x, blob, ws)
    torch.cuda.synchronize()
    return blob, blob.cpu().numpy(), ws


def gpu_decode(plan: B.Plan, blob_dev: torch.Tensor, tokens: int, ws: torch.Tensor, fill: float = 1.0) -> np.ndarray:
    y = torch.full((tokens, plan.hidden), fill, dtype=plan.dtype, device="cuda")
    plan.decode(blob_dev, tokens, y, ws)
    torch.cuda.synchronize()
    return synth.raw_u16(y.cpu())


def assert_blobs_equal(gpu_blob: np.ndarray, ref_blob: np.ndarray) -> None:
    """Bit-exact comparison of header and of every section up to the totals."""
    gh, rh = R.header(gpu_blob), R.header(ref_blob)
    assert gh == rh, (gh, rh)
    assert np.array_equal(gpu_blob[:64], ref_blob[:64])
    gs, rs = R.sections(gpu_blob), R.sections(ref_blob)
    for name in ("bits", "zp", "word_off", "out_ptr", "words", "outl"):
        if not np.array_equal(gs[name], rs[name]):
            bad = np.nonzero(gs[name] != rs[name])[0]
            raise AssertionError("section %s differs at %d places, first %s: gpu %s ref %s" % (
                name, bad.size, bad[:5], gs[name][bad[:5]], rs[name][bad[:5]]))
    assert np.array_equal(gs["scale"].view(np.uint32), rs["scale"].view(np.uint32)), "scale differs"


def full_parity(x_cpu: torch.Tensor, tau: float, bits, delta: float = 0.2, max_outliers: int = 0,
                plan: B.Plan = None, check_cross: bool = True, variant: int = 0):
    """Encode and decode on both sides; every byte must agree. Returns (gpu blob, reference blob)."""
    T, H = x_cpu.shape
    raw = synth.raw_u16(x_cpu)
    ref_blob = R.encode(raw, dt_code(x_cpu), tau, list(bits), delta, max_outliers, signed_values=variant == 1)
    if plan is None:
        plan = B.Plan(x_cpu.dtype, H, max(T, 1), tau, list(bits), delta, max_outliers, variant=variant)
    blob_dev, gpu_blob, ws = gpu_encode(plan, x_cpu)
    assert gpu_blob.size == ref_blob.size
    assert_blobs_equal(gpu_blob, ref_blob)
    info = plan.blob_info(blob_dev)
    rh = R.header(ref_blob)
    assert (info.status, info.tokens, info.hidden, info.total_words, info.total_outliers) == \
        (rh["status"], T, H, rh["total_words"], rh["total_outliers"])
    stored = min(rh["total_outliers"], rh["outlier_capacity"])
    assert info.payload_bytes == 64 + 9 * T + 8 * (T + 1) + 4 * rh["total_words"] + 4 * stored
    if rh["status"] == 0:
        ref_y = R.decode(ref_blob)
        y_gpu = gpu_decode(plan, blob_dev, T, ws)
        assert np.array_equal(y_gpu, ref_y), "decode differs at %d elements" % int((y_gpu != ref_y).sum())
        if check_cross:
            # GPU decode of the oracle's blob, oracle decode of the GPU's blob
            y_cross = gpu_decode(plan, torch.from_numpy(ref_blob).cuda(), T, ws)
            assert np.array_equal(y_cross, ref_y)
            assert np.array_equal(R.decode(gpu_blob), ref_y)
        assert plan.workspace_status(ws) == (0, 0)
    return gpu_blob, ref_blob
