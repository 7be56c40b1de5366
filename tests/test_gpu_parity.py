"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import tsq_ref as R
from paper_2511_04002_b200 import binding as B
from paper_2511_04002_b200 import synth
from tests._parity import assert_blobs_equal, full_parity, gpu_decode, gpu_encode

pytestmark = pytest.mark.gpu
INF = float("inf")


def rand16(shape, dtype, seed, scale=1.0, outlier_rate=0.0):
    g = torch.Generator().manual_seed(seed)
    v = torch.randn(shape, generator=g) * scale
    if outlier_rate > 0:
        hit = torch.rand(shape, generator=g) < outlier_rate
        v = torch.where(hit, v * 40, v)
    return v.to(dtype).contiguous()


# ------------------------------------------------------------------ tiny and ragged shapes

@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("shape", [(1, 8), (1, 32), (3, 40), (2, 4096), (5, 72), (7, 4104), (3, 264), (300, 8)])
def test_small_shapes(dtype, shape):
    x = rand16(shape, dtype, seed=shape[0] * 1000 + shape[1], scale=2.0, outlier_rate=0.02)
    full_parity(x, 6.0, [2, 4, 8], 0.2)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("delta", [-1.0, 0.0, 0.25, 0.5, 1.0, 1e9])
@pytest.mark.parametrize("bits", [[2, 4, 8], [2, 3, 4, 8], [2, 3, 4, 5, 6, 7, 8], [8], [3], [2, 5]])
def test_every_candidate_is_exercised(dtype, delta, bits):
    T, H = 48, 1024
    x = rand16((T, H), dtype, seed=len(bits) * 7 + int(delta * 4) % 5, scale=1.0, outlier_rate=0.001)
    # rows whose bulk is small against their range drop to low levels
    x[::3] = (x[::3].float().abs() ** 3 * 0.05).to(dtype) * torch.sign(x[::3].float()).to(dtype)
    gpu_blob, _ = full_parity(x, 6.0, bits, delta)
    chosen = set(R.sections(gpu_blob)["bits"].tolist())
    if delta >= 1e9:
        assert chosen == {bits[0]}
    if delta < 0:
        assert chosen == {bits[-1]}


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("shape", [(400, 10240), (330, 16384), (600, 8200), (700, 4104), (1000, 72), (450, 8192), (2000, 1024)])
def test_many_rows_take_the_pipelined_or_the_row_kernel(dtype, shape):
    # more rows than twice the SM count: rows of up to 8192 elements go through the pipelined kernel,
    # longer ones through the row-at-a-time kernel
    x = rand16(shape, dtype, seed=shape[0] * 1000 + shape[1], scale=2.0, outlier_rate=0.02)
    x[::7] = (x[::7].float().abs() ** 3 * 0.05).to(dtype) * torch.sign(x[::7].float()).to(dtype)   # rows that descend
    full_parity(x, 6.0, [2, 3, 4, 8], 0.2, check_cross=False)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("shape", [(500, 4096), (420, 8192), (900, 264)])
@pytest.mark.parametrize("delta", [0.2, 1e9])
def test_many_rows_some_needing_the_division_instruction(dtype, shape, delta):
    # the pipelined kernel's rolled path: rows whose zero-point is large (a narrow range far from zero) and,
    # for bf16, rows whose scale is far outside the range of the FMA quotient, among ordinary rows
    T, H = shape
    x = rand16(shape, dtype, seed=T * 31 + H, scale=1.5, outlier_rate=0.0).float()
    g = torch.Generator().manual_seed(T + H)
    x[::5] = 100.0 + torch.rand((x[::5].shape[0], H), generator=g)                    # zero-point 12700: past the packed steps
    x[4::5] = 100.0 + torch.rand((x[4::5].shape[0], H), generator=g) * 0.0625         # fp16: zero-point 203200; bf16: a constant row
    x[1::5] = -(3.0 + torch.rand((x[1::5].shape[0], H), generator=g) * 0.25)          # zero-point of a few thousand: packed steps
    if dtype == torch.bfloat16:
        x[2::11] *= 1e37
        x[3::13] *= 1e-36
    full_parity(x.to(dtype).contiguous(), INF, [2, 3, 4, 8], delta, check_cross=False)


@pytest.mark.parametrize("case", range(24))
def test_randomized_many_row_cases(case):
    # seeded draws over the shapes, candidate sets, thresholds and tolerances that select between the kernels
    # and between their paths (whole and ragged groups, descent depth, outlier lists that overflow)
    rng = np.random.default_rng(1000 + case)
    H = int(rng.choice([8, 72, 264, 1024, 2048, 4096, 4104, 5120, 8192, 8184])) if rng.random() < 0.7 else int(rng.integers(1, 1025)) * 8
    T = int(rng.integers(297, 1400))
    if T * H > 6_000_000:
        T = max(297, 6_000_000 // H)
    dtype = torch.float16 if rng.random() < 0.5 else torch.bfloat16
    g = torch.Generator().manual_seed(int(rng.integers(1 << 30)))
    scale = float(rng.choice([0.3, 1.0, 2.0, 5.0]))
    v = torch.randn((T, H), generator=g) * scale * torch.exp(torch.randn((T, 1), generator=g) * 0.5)
    if rng.random() < 0.5:
        v = torch.where(torch.rand((T, H), generator=g) < 0.01, v * 30, v)
    bits = [[2, 4, 8], [2, 3, 4, 8], [8], [3, 5], [2, 3, 4, 5, 6, 7, 8]][int(rng.integers(5))]
    delta = float(rng.choice([0.2, 0.0, 0.5, 1e9, -1.0]))
    tau = float(rng.choice([6.0, 1.0, 3.0, INF]))
    full_parity(v.to(dtype).contiguous(), tau, bits, delta, check_cross=False)


@pytest.mark.parametrize("hidden", [16384, 65536])
def test_long_rows(hidden):
    x = rand16((5, hidden), torch.bfloat16, seed=hidden, scale=1.5, outlier_rate=0.001)
    full_parity(x, 6.0, [2, 4, 8], 0.2)


# ------------------------------------------------------------------ adversarial rows

def _special_rows(dtype, H=256):
    rows = []
    z = torch.zeros(H)
    rows.append(z.clone())                                   # all zero
    rows.append(torch.full((H,), 2.5))                       # constant
    rows.append(torch.full((H,), -3.0))                      # constant negative
    r = torch.randn(H); r[0] = 0.0; r[1] = -0.0; rows.append(r)
    r = torch.randn(H) * 100; rows.append(r)                 # mostly outliers
    r = torch.randn(H) * 0.01; rows.append(r)                # no outliers
    r = torch.randn(H); r[3] = float("nan"); r[5] = INF; r[7] = -INF; rows.append(r)
    r = torch.randn(H); r[10] = 6.0; r[11] = -6.0; r[12] = 5.99; rows.append(r)      # |x| == tau
    r = (torch.arange(H) % 9).float() * 0.5; rows.append(r)  # many exact .5 ties in m / s
    r = torch.arange(H).float() / H + 100.0; rows.append(r)  # narrow range far from zero -> large zero-point
    r = torch.ones(H) * 4; r[0] = 4.004; rows.append(r)      # two adjacent values
    r = torch.randn(H).abs() + 1.0; rows.append(r)           # non-zero minimum
    x = torch.stack(rows).to(dtype)
    # subnormal rows, built from raw patterns
    sub = torch.zeros((2, H), dtype=dtype)
    raw = synth.raw_u16(sub).copy()
    rng = np.random.default_rng(1)
    raw[0] = rng.integers(0, 0x0400 if dtype == torch.float16 else 0x0080, H).astype(np.uint16)
    raw[1] = rng.integers(0, 0x0400 if dtype == torch.float16 else 0x0080, H).astype(np.uint16) | \
        (rng.integers(0, 2, H).astype(np.uint16) << 15)
    raw[1, ::5] = 0x3c00 if dtype == torch.float16 else 0x3f80   # subnormals next to 1.0
    sub = synth.from_raw_u16(raw, "f16" if dtype == torch.float16 else "bf16")
    return torch.cat([x, sub]).contiguous()


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("tau", [6.0, INF, 0.0, -1.0, 1e-7, 70000.0])
def test_special_rows(dtype, tau):
    full_parity(_special_rows(dtype), tau, [2, 4, 8], 0.2)
    full_parity(_special_rows(dtype), tau, [2, 3, 4, 5, 6, 7, 8], 0.5)


def test_huge_and_tiny_bf16_scales():
    H = 512
    g = torch.Generator().manual_seed(9)
    big = (torch.randn((4, H), generator=g) * 1e37).to(torch.bfloat16)       # scale above 2^100
    tiny = (torch.randn((4, H), generator=g) * 1e-36).to(torch.bfloat16)     # scale below 2^-100
    x = torch.cat([big, tiny]).contiguous()
    full_parity(x, INF, [2, 4, 8], 0.2)
    full_parity(x, 1e30, [4, 8], 1.0)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_all_16bit_magnitudes_appear(dtype):
    # every finite non-negative pattern, shuffled into rows, so each rounding boundary meets a real value
    top = 0x7c00 if dtype == torch.float16 else 0x7f80
    pats = np.arange(top, dtype=np.uint32).astype(np.uint16)
    rng = np.random.default_rng(0)
    H = 1024
    rows = []
    for lo_exp in range(0, top, 2048):
        seg = pats[lo_exp:lo_exp + 2048].copy()
        rng.shuffle(seg)
        rows.append(seg[:H]); rows.append(seg[H:2 * H] if seg.size >= 2 * H else np.resize(seg, H))
    raw = np.stack(rows)
    raw |= (rng.integers(0, 2, raw.shape).astype(np.uint16) << 15)
    x = synth.from_raw_u16(raw, "f16" if dtype == torch.float16 else "bf16")
    full_parity(x, INF, [2, 3, 4, 5, 6, 7, 8], 0.3)


# ------------------------------------------------------------------ the paper-shaped workloads

def test_c1_prefill():
    w = synth.c1_prefill()
    full_parity(synth.make(w), w.tau, w.bits, w.delta)


def test_c2_all_decode_steps_share_one_workspace():
    w = synth.c2_decode_steps()                      # all 512 steps of the workload, one plan, one workspace, one blob
    plan = B.Plan(torch.float16, w.recipe.hidden, w.recipe.tokens, w.tau, list(w.bits), w.delta)
    blob, ws = plan.alloc()
    for i in range(w.steps):
        x = synth.make(w, i)
        ref = R.encode(synth.raw_u16(x), R.F16, w.tau, list(w.bits), w.delta)
        _, got, _ = gpu_encode(plan, x, ws=ws, blob=blob)
        assert_blobs_equal(got, ref)
        assert np.array_equal(gpu_decode(plan, blob, w.recipe.tokens, ws), R.decode(ref))
    assert plan.workspace_status(ws) == (0, 0)


def test_c3_13b_prefill():
    w = synth.c3_13b_prefill()
    full_parity(synth.make(w), w.tau, w.bits, w.delta, check_cross=False)


def test_c4_70b_prefill_reduced():
    w = synth.c4_70b_prefill(tokens=768)
    full_parity(synth.make(w), w.tau, w.bits, w.delta, check_cross=False)


@pytest.mark.parametrize("w", [8, 256])
def test_kv_cache_workload(w):
    wl = synth.kv_cache(w)
    x = synth.make(wl)
    gpu_blob, _ = full_parity(x, wl.tau, wl.bits, wl.delta, check_cross=False)
    assert R.header(gpu_blob)["total_outliers"] > 0


@pytest.mark.parametrize("i_tok", [0, 1, 2, 3, 4])
@pytest.mark.parametrize("i_rate", [0, 1, 2])
@pytest.mark.parametrize("i_dtype", [0, 1])
def test_c5_sweep(i_tok, i_rate, i_dtype):
    # every point of the sweep, the 4096- and 32768-token ones included, every byte compared
    w = synth.c5_sweep_point(i_tok, i_rate, i_dtype)
    full_parity(synth.make(w), w.tau, w.bits, w.delta, check_cross=False)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_long_rows_with_few_and_very_many_outliers_mixed(dtype):
    # hidden 8192, more rows than a persistent CTA keeps in flight many times over, and rows with 0, 1, about 600
    # and about 4000 outliers next to one another: the rows whose outliers do not fit a CTA's list are placed
    # while ordinary rows queue behind them
    T, H = 3100, 8192
    g = torch.Generator().manual_seed(77)
    v = torch.randn((T, H), generator=g)
    kind = torch.randint(0, 4, (T,), generator=g)
    for t in range(T):
        k = int(kind[t])
        if k == 1:
            v[t, int(torch.randint(0, H, (1,), generator=g))] = 50.0
        elif k >= 2:
            n = 600 if k == 2 else 4000
            cols = torch.randperm(H, generator=g)[:n]
            v[t, cols] = torch.where(torch.rand(n, generator=g) < 0.5, -1.0, 1.0) * (20.0 + 60.0 * torch.rand(n, generator=g))
    x = v.to(dtype).contiguous()
    counts = (~(x.float().abs() < 6.0)).sum(dim=1)
    assert int((counts == 0).sum()) > 100 and int((counts == 1).sum()) > 100
    assert int(((counts > 500) & (counts < 700)).sum()) > 100 and int((counts > 3900).sum()) > 100
    full_parity(x, 6.0, [2, 4, 8], 0.2, check_cross=False)


@pytest.mark.parametrize("hidden,max_outliers", [(4096, 0), (5120, 0), (1000, 0), (4096, 300000)])
def test_runs_of_rows_that_are_mostly_outliers(hidden, max_outliers):
    # every persistent CTA meets several rows in a row whose outliers exceed its lists (a third to all of the row),
    # between stretches of ordinary rows; the last case also runs out of CSR capacity in the middle of such a row
    T = 1500
    g = torch.Generator().manual_seed(hidden)
    v = torch.randn((T, hidden), generator=g)
    v[300:900] *= torch.linspace(4.0, 40.0, 600).unsqueeze(1)
    v[1200:1230] *= 100.0
    x = v.to(torch.float16).contiguous()
    counts = (~(x.float().abs() < 6.0)).sum(dim=1)
    assert int((counts > hidden // 3).sum()) > 500 and int((counts == 0).sum()) > 100
    gpu_blob, _ = full_parity(x, 6.0, [2, 4, 8], 0.2, max_outliers=max_outliers, check_cross=False)
    assert R.header(gpu_blob)["status"] == (6 if max_outliers else 0)


# ------------------------------------------------------------------ asynchronous conditions and errors

def test_outlier_overflow_is_reported():
    x = rand16((6, 512), torch.float16, seed=3, scale=3.0, outlier_rate=0.05)
    gpu_blob, ref_blob = full_parity(x, 6.0, [2, 4, 8], 0.2, max_outliers=10)
    assert R.header(gpu_blob)["status"] == 6
    plan = B.Plan(torch.float16, 512, 6, 6.0, [2, 4, 8], 0.2, 10)
    blob, _, ws = gpu_encode(plan, x)
    assert plan.workspace_status(ws)[0] == 6
    y = gpu_decode(plan, blob, 6, ws, fill=1.0)              # decoder refuses the blob, writes nothing
    assert np.all(y == synth.raw_u16(torch.ones(1, dtype=torch.float16))[0])
    assert plan.workspace_status(ws)[1] == 6
    plan.workspace_init(ws)
    x2 = rand16((6, 512), torch.float16, seed=4, scale=0.5)
    _, got, _ = gpu_encode(plan, x2, ws=ws, blob=blob)       # the same buffers work again
    assert_blobs_equal(got, R.encode(synth.raw_u16(x2), R.F16, 6.0, [2, 4, 8], 0.2, 10))


def test_decoder_rejects_corrupt_blobs_without_writing():
    x = rand16((4, 256), torch.float16, seed=5, scale=1.0, outlier_rate=0.01)
    plan = B.Plan(torch.float16, 256, 4, 6.0, [2, 4, 8], 0.2)
    blob, host, ws = gpu_encode(plan, x)
    one = synth.raw_u16(torch.ones(1, dtype=torch.float16))[0]
    lay = R.layout(256, 4, 8, 0)
    cases = []
    b = host.copy(); b[0] ^= 0xff; cases.append(b)                                 # magic
    b = host.copy(); b[16] = 3; cases.append(b)                                    # tokens in header
    b = host.copy(); b[lay["bits"] + 1] = 9; cases.append(b)                       # bit-width out of range
    b = host.copy(); b[lay["word_off"] + 4:lay["word_off"] + 8] = 255; cases.append(b)   # offset out of range
    b = host.copy(); b[lay["out_ptr"] + 8:lay["out_ptr"] + 12] = 255; cases.append(b)    # CSR pointer out of range
    for bad in cases:
        plan.workspace_init(ws)
        y = gpu_decode(plan, torch.from_numpy(bad).cuda(), 4, ws, fill=1.0)
        assert plan.workspace_status(ws)[1] == 5
        changed_rows = np.nonzero((y != one).any(axis=1))[0]
        assert changed_rows.size < 4                          # the offending rows (or all of them) are untouched
    plan.workspace_init(ws)
    y = gpu_decode(plan, blob, 4, ws)
    assert plan.workspace_status(ws) == (0, 0)
    assert np.array_equal(y, R.decode(host))


def test_argument_errors_are_synchronous():
    plan = B.Plan(torch.float16, 256, 4, 6.0, [2, 4, 8], 0.2)
    blob, ws = plan.alloc()
    x = torch.zeros((4, 256), dtype=torch.float16, device="cuda")
    with pytest.raises(B.TsqError) as e:
        plan.encode(x, blob[:128], ws)
    assert e.value.status == 3
    with pytest.raises(B.TsqError) as e:
        plan.encode(x, blob, ws[:32])
    assert e.value.status == 3
    with pytest.raises(B.TsqError) as e:
        plan.encode(torch.zeros((5, 256), dtype=torch.float16, device="cuda"), blob, ws)
    assert e.value.status == 1
    with pytest.raises(B.TsqError) as e:
        plan.encode(x, blob[8:], ws)                          # misaligned blob
    assert e.value.status == 1
    for bad in ([], [1, 4], [4, 4], [2, 9]):
        with pytest.raises(B.TsqError):
            B.Plan(torch.float16, 256, 4, 6.0, bad)
    with pytest.raises(B.TsqError) as e:
        B.Plan(torch.float16, 100, 4, 6.0, [2, 4])
    assert e.value.status == 2


def test_empty_call_writes_a_valid_blob():
    plan = B.Plan(torch.bfloat16, 512, 16, 6.0, [2, 4, 8], 0.2)
    blob, ws = plan.alloc(0)
    blob.fill_(0xA5)                                      # what a sender would ship must not be left over
    x = torch.zeros((0, 512), dtype=torch.bfloat16, device="cuda")
    plan.encode(x, blob, ws)
    torch.cuda.synchronize()
    ref = R.encode(np.zeros((0, 512), np.uint16), R.BF16, 6.0, [2, 4, 8], 0.2)
    got = blob.cpu().numpy()
    assert np.array_equal(got[:64], ref[:64])
    assert_blobs_equal(got, ref)                          # word_off[0] and out_ptr[0] included
    assert plan.blob_info(blob).payload_bytes == 64 + 8
    y = torch.zeros((0, 512), dtype=torch.bfloat16, device="cuda")
    plan.decode(blob, 0, y, ws)
    # the plan still serves a non-empty call afterwards, with the same workspace size
    blob2, ws2 = plan.alloc(16)
    xs = rand16((16, 512), torch.bfloat16, seed=8)
    _, got, _ = gpu_encode(plan, xs, ws=ws2, blob=blob2)
    assert_blobs_equal(got, R.encode(synth.raw_u16(xs), R.BF16, 6.0, [2, 4, 8], 0.2))


def test_run_to_run_determinism_and_host_calls():
    w = synth.c5_sweep_point(2, 2, 1)
    x = synth.make(w)
    plan = B.Plan(x.dtype, w.recipe.hidden, w.recipe.tokens, w.tau, list(w.bits), w.delta)
    blob, ws = plan.alloc()
    _, a, _ = gpu_encode(plan, x, ws=ws, blob=blob)
    blob.zero_()
    _, b, _ = gpu_encode(plan, x, ws=ws, blob=blob)
    assert_blobs_equal(a, b)
    # host-buffer entry points: same bytes as the device calls
    T = w.recipe.tokens
    x_pin = x.pin_memory()
    blob_host = torch.zeros(blob.numel(), dtype=torch.uint8).pin_memory()
    x_dev = torch.empty_like(x, device="cuda")
    payload = plan.encode_host(x_pin, blob_host, x_dev, blob, ws)
    assert payload == plan.blob_info(blob).payload_bytes
    assert_blobs_equal(blob_host.numpy(), a)
    y_host = torch.empty_like(x).pin_memory()
    y_dev = torch.empty_like(x, device="cuda")
    plan.decode_host(blob_host, T, y_host, blob, y_dev, ws)
    assert np.array_equal(synth.raw_u16(y_host), R.decode(a))


# ------------------------------------------------------------------ full size, as the benchmark launches it

def test_c4_full_size_every_byte_and_invariants():
    """The benchmark's workload at its full size (8192 x 8192 bf16), same plan and launch shape: every section of
    the blob and every element of the reconstruction against the oracle, plus properties that hold at any size
    (checked independently of the oracle)."""
    w = synth.c4_70b_prefill()
    x = synth.make(w)
    T, H = x.shape
    plan = B.Plan(x.dtype, H, T, w.tau, list(w.bits), w.delta)
    host, _ = full_parity(x, w.tau, w.bits, w.delta, plan=plan, check_cross=False)
    hdr, sec = R.header(host), R.sections(host)
    wpp = H // 32
    raw = synth.raw_u16(x)
    # placement: plain prefix sums, outlier counts equal an independent count of |x| >= tau (NaN/Inf included)
    assert np.array_equal(sec["word_off"], np.concatenate([[0], np.cumsum(sec["bits"].astype(np.int64) * wpp)]))
    out = ~(x.float().abs() < w.tau)
    assert np.array_equal(np.diff(sec["out_ptr"].astype(np.int64)), out.sum(dim=1).numpy())
    assert hdr["total_words"] == int(sec["word_off"][-1]) and hdr["total_outliers"] == int(sec["out_ptr"][-1])
    # CSR: ascending columns per row, original patterns
    rows_of = np.repeat(np.arange(T), np.diff(sec["out_ptr"].astype(np.int64)))
    cols = (sec["outl"] >> 16).astype(np.int64)
    assert np.array_equal(raw[rows_of, cols], (sec["outl"] & 0xffff).astype(np.uint16))
    same_row = rows_of[1:] == rows_of[:-1]
    assert np.all(cols[1:][same_row] > cols[:-1][same_row])
