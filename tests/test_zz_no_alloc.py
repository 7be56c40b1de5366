"""tsq_encode_noalloc against tsq_encode.

Some callers of the codec may not allocate device memory at the point where they encode (a serving
loop that runs with a frozen memory pool, a plug-in inside a runtime that owns all device memory).
For them the library keeps the encoder's look-back scratch in a fixed array of its own.  This test
calls that entry point through the C ABI and requires the very same blob, byte for byte over every
meaningful section, as the ordinary entry point gives with a caller-allocated workspace: twice in a
row on different inputs, because the second call meets the first call's leftovers in the shared array.
"""
import numpy as np
import pytest
import torch

from oracle import tsq_ref as R
from paper_2511_04002_b200 import binding as B
from paper_2511_04002_b200 import synth
from tests._parity import assert_blobs_equal

pytestmark = pytest.mark.gpu


def _input(seed, tokens, hidden, dtype):
    g = torch.Generator().manual_seed(seed)
    v = torch.randn((tokens, hidden), generator=g) * 1.5
    hit = torch.rand((tokens, hidden), generator=g) < 0.003
    return torch.where(hit, v * 30, v).to(dtype).contiguous()


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_noalloc_matches_workspace_encode_twice(dtype):
    hidden, max_tokens = 2048, 300
    plan = B.Plan(dtype, hidden, max_tokens, 6.0, [2, 4, 8], 0.2)
    blob_ref, ws = plan.alloc(max_tokens)
    for call, tokens in enumerate((300, 173)):            # the second call is shorter: stale entries lie beyond it
        x = _input(100 + call, tokens, hidden, dtype).cuda()
        blob_bytes, _ = plan.sizes(tokens)
        blob_new = torch.zeros(blob_bytes, dtype=torch.uint8, device="cuda")
        plan.encode(x, blob_ref, ws)
        plan.encode_noalloc(x, blob_new)
        torch.cuda.synchronize()
        info = plan.blob_info(blob_new)
        assert info.status == 0 and info.tokens == tokens
        got, want = blob_new.cpu().numpy(), blob_ref.cpu().numpy()
        assert_blobs_equal(got, want)
        # and it decodes to the oracle's reconstruction of the oracle's own blob
        y = torch.empty_like(x)
        plan.decode(blob_new, tokens, y, ws)
        torch.cuda.synchronize()
        code = R.F16 if dtype == torch.float16 else R.BF16
        ref_blob = R.encode(synth.raw_u16(x.cpu()), code, 6.0, [2, 4, 8], 0.2)
        assert np.array_equal(synth.raw_u16(y.cpu()), R.decode(ref_blob))


def test_noalloc_refuses_plans_beyond_its_scratch():
    plan = B.Plan(torch.float16, 256, 16385, 6.0, [2, 4, 8], 0.2)
    blob_bytes, _ = plan.sizes(4)
    blob = torch.zeros(blob_bytes, dtype=torch.uint8, device="cuda")
    x = torch.zeros((4, 256), dtype=torch.float16, device="cuda")
    with pytest.raises(B.TsqError) as e:
        plan.encode_noalloc(x, blob)
    assert e.value.status == 2                             # TSQ_ERR_UNSUPPORTED, nothing was enqueued
    assert not blob.any()
