"""GPU parity of the signed-values variant (Eq. "Proposed" on the signed inliers, Q_max = 2^b - 1, no sign
plane): the CUDA path through the C ABI against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import tsq_ref as R
from paper_2511_04002_b200 import binding as B
from paper_2511_04002_b200 import synth
from tests._parity import full_parity, gpu_encode
from tests.test_gpu_parity import _special_rows, rand16

pytestmark = pytest.mark.gpu
INF = float("inf")
SV = B.VARIANT_SIGNED_VALUES


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("shape", [(1, 8), (1, 32), (3, 40), (2, 4096), (5, 72), (7, 4104), (3, 264), (300, 8)])
def test_small_shapes(dtype, shape):
    x = rand16(shape, dtype, seed=shape[0] * 1000 + shape[1] + 1, scale=2.0, outlier_rate=0.02)
    full_parity(x, 6.0, [2, 4, 8], 0.2, variant=SV)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("delta", [-1.0, 0.0, 0.25, 0.5, 1.0, 1e9])
@pytest.mark.parametrize("bits", [[2, 4, 8], [2, 3, 4, 5, 6, 7, 8], [8], [3], [2, 5]])
def test_every_candidate_is_exercised(dtype, delta, bits):
    T, H = 48, 1024
    x = rand16((T, H), dtype, seed=len(bits) * 7 + int(delta * 4) % 5 + 50, scale=1.0, outlier_rate=0.001)
    x[::3] = (x[::3].float().abs() ** 3 * 0.05).to(dtype) * torch.sign(x[::3].float()).to(dtype)
    x[1::6] = x[1::6].abs()                                  # non-negative rows
    x[2::6] = -x[2::6].abs() - 1                             # rows below zero: negative zero-points
    gpu_blob, _ = full_parity(x, 6.0, bits, delta, variant=SV)
    sec = R.sections(gpu_blob)
    chosen = set(sec["bits"].tolist())
    if delta >= 1e9:
        assert chosen == {bits[0]}
    if delta < 0:
        assert chosen == {bits[-1]}
    assert (sec["zp"] < 0).any()


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("shape", [(400, 10240), (330, 16384), (700, 4104), (1000, 72), (450, 8192), (2000, 1024)])
def test_many_rows_are_handed_out_by_ticket(dtype, shape):
    x = rand16(shape, dtype, seed=shape[0] * 1000 + shape[1] + 2, scale=2.0, outlier_rate=0.02)
    x[::7] = (x[::7].float().abs() ** 3 * 0.05).to(dtype) * torch.sign(x[::7].float()).to(dtype)
    x[3::7] = x[3::7].abs()                                  # non-negative rows
    # (a row spread around zero seldom passes the distortion test here: its codes sit mid-range, where the 8-bit
    # code shifted right and the lower level's code differ by the ratio 255/16 : 15, so a second tolerance joins in)
    for delta in (0.2, 0.4):
        gpu_blob, _ = full_parity(x, 6.0, [2, 3, 4, 8], delta, check_cross=False, variant=SV)
    assert len(set(R.sections(gpu_blob)["bits"].tolist())) > 1


@pytest.mark.parametrize("hidden", [16384, 40000, 65536])
def test_long_rows(hidden):
    x = rand16((5, hidden), torch.bfloat16, seed=hidden + 3, scale=1.5, outlier_rate=0.001)
    full_parity(x, 6.0, [2, 4, 8], 0.2, variant=SV)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("tau", [6.0, INF, 0.0, -1.0, 1e-7, 70000.0])
def test_special_rows(dtype, tau):
    full_parity(_special_rows(dtype), tau, [2, 4, 8], 0.2, variant=SV)
    full_parity(_special_rows(dtype), tau, [2, 3, 4, 5, 6, 7, 8], 0.5, variant=SV)
    full_parity(-_special_rows(dtype), tau, [2, 3, 4, 8], 0.5, variant=SV)


def test_huge_and_tiny_bf16_scales():
    H = 512
    g = torch.Generator().manual_seed(19)
    big = (torch.randn((4, H), generator=g) * 1e37).to(torch.bfloat16)
    tiny = (torch.randn((4, H), generator=g) * 1e-36).to(torch.bfloat16)
    x = torch.cat([big, tiny]).contiguous()
    full_parity(x, INF, [2, 4, 8], 0.2, variant=SV)
    full_parity(x, 1e30, [4, 8], 1.0, variant=SV)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_all_finite_16bit_patterns_appear(dtype):
    # every finite pattern of either sign, shuffled into rows, so each rounding boundary meets a real value
    top = 0x7c00 if dtype == torch.float16 else 0x7f80
    pats = np.concatenate([np.arange(top, dtype=np.uint32), np.arange(top, dtype=np.uint32) | 0x8000]).astype(np.uint16)
    rng = np.random.default_rng(3)
    H = 1024
    rows = []
    for lo in range(0, top, 2048):                           # rows of similar magnitude, both signs
        seg = np.concatenate([pats[lo:lo + 2048], pats[top + lo:top + lo + 2048]])
        rng.shuffle(seg)
        for k in range(0, seg.size - H + 1, H):
            rows.append(seg[k:k + H])
    raw = np.stack(rows)
    x = synth.from_raw_u16(raw, "f16" if dtype == torch.float16 else "bf16")
    full_parity(x, INF, [2, 3, 4, 5, 6, 7, 8], 0.3, variant=SV)


def test_c1_and_c3_workloads():
    for w in (synth.c1_prefill(), synth.c3_13b_prefill()):
        full_parity(synth.make(w), w.tau, w.bits, w.delta, check_cross=False, variant=SV)


def test_runs_of_rows_that_are_mostly_outliers():
    # rows whose outliers exceed a persistent CTA's lists, several in a row, between stretches of ordinary rows
    T, H = 1200, 4096
    g = torch.Generator().manual_seed(4096)
    v = torch.randn((T, H), generator=g)
    v[300:800] *= torch.linspace(4.0, 40.0, 500).unsqueeze(1)
    full_parity(v.to(torch.bfloat16).contiguous(), 6.0, [2, 4, 8], 0.2, check_cross=False, variant=SV)


def test_c4_shaped_rows():
    w = synth.c4_70b_prefill(1024)
    full_parity(synth.make(w), w.tau, w.bits, w.delta, check_cross=False, variant=SV)


def test_outlier_overflow_is_reported():
    x = rand16((40, 512), torch.float16, seed=77, scale=3.0, outlier_rate=0.05)
    raw = synth.raw_u16(x)
    ref = R.encode(raw, R.F16, 6.0, [2, 4, 8], 0.2, 100, signed_values=True)
    assert R.header(ref)["status"] == 6
    plan = B.Plan(torch.float16, 512, 40, 6.0, [2, 4, 8], 0.2, 100, variant=SV)
    blob_dev, gpu_blob, ws = gpu_encode(plan, x)
    assert plan.blob_info(blob_dev).status == 6 and R.header(gpu_blob)["total_outliers"] == R.header(ref)["total_outliers"]


def test_a_plan_of_the_other_variant_rejects_the_blob():
    x = rand16((9, 256), torch.float16, seed=5)
    plan_sv = B.Plan(torch.float16, 256, 9, 6.0, [2, 4, 8], 0.2, variant=SV)
    plan_m = B.Plan(torch.float16, 256, 9, 6.0, [2, 4, 8], 0.2)
    for enc, dec in ((plan_sv, plan_m), (plan_m, plan_sv)):
        blob_dev, _, ws = gpu_encode(enc, x)
        y = torch.full((9, 256), 7.0, dtype=torch.float16, device="cuda")
        dec.decode(blob_dev, 9, y, ws)
        torch.cuda.synchronize()
        assert dec.workspace_status(ws)[1] == 5
        assert bool((y == 7.0).all())


def test_unknown_variant_is_an_argument_error():
    with pytest.raises(B.TsqError) as e:
        B.Plan(torch.float16, 256, 9, 6.0, [2, 4, 8], 0.2, variant=2)
    assert e.value.status == 1
