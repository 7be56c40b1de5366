"""The seeded input generator (no GPU): determinism, shapes and the structure each recipe promises."""
import numpy as np
import torch

from paper_2511_04002_b200 import synth


def test_same_seed_same_bytes_and_steps_differ():
    w = synth.c2_decode_steps(4)
    a, b = synth.make(w, 0), synth.make(w, 0)
    assert a.dtype == torch.float16 and a.shape == (64, 4096)
    assert np.array_equal(synth.raw_u16(a), synth.raw_u16(b))
    assert not np.array_equal(synth.raw_u16(a), synth.raw_u16(synth.make(w, 1)))


def test_c1_has_its_fixed_outlier_channels():
    w = synth.c1_prefill()
    x = synth.make(w).float()
    big = (x.abs() >= w.tau).float().mean(0)                   # per channel: share of tokens above tau
    assert int((big > 0.5).sum()) == 8                         # the eight channels times 50
    assert float(big.sort().values[:-8].max()) < 0.2


def test_kv_cache_rows_are_layers_of_keys_then_values():
    w = synth.kv_cache(w=16, layers=6)
    x = synth.make(w).float()
    assert x.shape == (2 * 6 * 16, 4096) and w.recipe.kv_layers == 6
    blocks = x.reshape(12, 16, 4096)                           # [layer][key | value] blocks of w rows
    col_rms = blocks.pow(2).mean(1).sqrt()                     # [12, 4096]
    ratio = col_rms / col_rms.median(1, keepdim=True).values
    heavy = ratio > 4.0
    assert all(int(heavy[k].sum()) == 8 for k in range(0, 12, 2))      # key blocks: the eight channels times 8
    assert all(int(heavy[k].sum()) == 0 for k in range(1, 12, 2))      # value blocks: none
    assert torch.equal(heavy[0], heavy[2])                              # the same channels in every layer
    scales = col_rms.median(1).values
    assert float(scales.max() / scales.min()) > 1.2                    # layers differ in scale
