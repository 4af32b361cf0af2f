"""The synthetic input generators: deterministic, slab independent, right shapes."""
import numpy as np
import torch

from paper_2510_23938_b200 import inputs


def test_uniform_bytes_are_deterministic_and_prefix_stable():
    a = inputs.uniform_bytes(1000, seed=1)
    b = inputs.uniform_bytes(1000, seed=1)
    c = inputs.uniform_bytes(1003, seed=1)
    assert torch.equal(a, b) and torch.equal(a, c[:1000])
    assert not torch.equal(a, inputs.uniform_bytes(1000, seed=2))
    assert 110 < float(a.float().mean()) < 145


def test_bf16_normal_statistics_and_piecewise_generation():
    w = inputs.bf16_normal_bytes(200_000, seed=3)
    v = w.view(torch.bfloat16).float()
    assert abs(v.mean().item()) < 5e-4 and abs(v.std().item() - 0.02) < 5e-4
    part = torch.empty(2 * 1000, dtype=torch.uint8)
    inputs.fill_bf16_normal(part, seed=3, first_elem=500)
    assert torch.equal(part, w[1000:3000])


def test_weight_file_layout_is_self_consistent():
    import json
    import struct
    blob, table = inputs.weight_file(inputs.tiny_tensors(), seed=7)
    raw = blob.numpy().tobytes()
    (hlen,) = struct.unpack("<Q", raw[:8])
    index = json.loads(raw[8:8 + hlen])
    assert len(index) == len(table)
    end = 0
    for name, off, nbytes in table:
        lo, hi = index[name]["data_offsets"]
        assert off == 8 + hlen + lo and nbytes == hi - lo
        end = max(end, off + nbytes)
    assert end == len(raw)


def test_model_shapes_match_the_named_workloads():
    _, t13, total13 = inputs.weight_file_layout(inputs.gpt_1p3b_tensors())
    assert 2.6e9 < total13 < 2.7e9
    _, t8, total8 = inputs.weight_file_layout(inputs.llama_8b_tensors())
    assert len(t8) == 291
    assert sum(n for _, _, n in t8) == 2 * 8_030_261_248
    assert -(-total8 // (4 << 20)) == 3830


def test_ragged_sizes_are_log_uniform_in_range():
    s = inputs.ragged_sizes()
    assert s.shape == (10_000,) and s.min() >= 4096 and s.max() <= 64 << 20 and (s % 2 == 0).all()
    logs = np.log(s.astype(np.float64))
    assert abs(np.median(logs) - (np.log(4096) + np.log(64 << 20)) / 2) < 0.15
    off = inputs.packed_offsets(s, first=6)
    assert off[0] == 6 and (np.diff(off) == s[:-1]).all()
