"""The seeded input generator: device independent, order independent, right distribution."""
import numpy as np
import pytest
import torch

from paper_2510_04147_b200 import workloads as wl


def test_hash_matches_pure_python():
    idx = torch.tensor([0, 1, 2, 12345, 2**31 + 7, 2**40 + 3], dtype=torch.int64)
    got = wl.hash_u64(7, 3, idx).tolist()
    for i, g in zip(idx.tolist(), got):
        assert (g & ((1 << 64) - 1)) == wl.hash_u64_py(7, 3, i)


def test_normal_tensor_statistics_and_chunking():
    a = wl.normal_tensor(1, 5, (1000, 300), 0.02)
    assert abs(a.mean().item()) < 2e-4
    assert abs(a.std().item() - 0.02) < 2e-4
    k = ((a / 0.02) ** 4).mean().item()
    assert abs(k - 3.0) < 0.1                          # normal kurtosis
    b = wl.normal_tensor(1, 5, (1000, 300), 0.02, chunk=7777)
    assert torch.equal(a, b)
    c = wl.normal_tensor(1, 6, (1000, 300), 0.02)
    assert not torch.equal(a, c)
    assert abs(np.corrcoef(a.flatten().numpy(), c.flatten().numpy())[0, 1]) < 0.01


def test_prompts_never_mask_and_batch_prefix_stable():
    w = wl.LLADA_8B
    p8 = wl.make_prompts(w, batch=8)
    p1 = wl.make_prompts(w, batch=1)
    assert p8.shape == (8, 512) and p8.dtype == torch.int32
    assert torch.equal(p8[:1], p1)
    assert int(p8.max()) < w.mask_id and int(p8.min()) >= 0
    assert len(torch.unique(p8)) > 3500


def test_tensor_specs_parameter_counts():
    """Layer / LM-head parameter counts of the two large shapes (they set the bytes per forward)."""
    def count(w, pred):
        n = 0
        for name, shape, _ in wl.tensor_specs(w):
            if pred(name):
                n += shape[0] * shape[1]
        return n
    assert count(wl.LLADA_8B, lambda n: n.startswith("layers.")) == 6_979_321_856
    assert count(wl.LLADA_8B, lambda n: n == "lm_head") == 517_996_544
    assert count(wl.DREAM_7B, lambda n: n.startswith("layers.")) == 6_525_288_448
    assert count(wl.DREAM_7B, lambda n: n == "lm_head") == 544_997_376


def test_make_tensor_dtype_and_determinism():
    t = wl.make_tensor(wl.TINY, "layers.1.w_down")
    assert t.dtype == torch.float32 and t.shape == (256, 688)
    assert torch.equal(t, wl.make_tensor(wl.TINY, "layers.1.w_down"))
    g = wl.make_tensor(wl.TINY, "norm_final")
    assert torch.equal(g, torch.ones(256))
    small = wl.LLADA_8B.replace(n_layers=1, vocab=512, d_model=128, d_ffn=256, n_heads=1, n_kv_heads=1)
    assert wl.make_tensor(small, "lm_head").dtype == torch.bfloat16


@pytest.mark.gpu
def test_generator_is_device_independent():
    w = wl.TINY
    for name in ("embed", "layers.0.wq", "lm_head"):
        assert torch.equal(wl.make_tensor(w, name, "cpu"), wl.make_tensor(w, name, "cuda").cpu())
    wb = wl.LLADA_8B.replace(n_layers=1, vocab=4096)
    assert torch.equal(wl.make_tensor(wb, "layers.0.w_gate", "cpu"), wl.make_tensor(wb, "layers.0.w_gate", "cuda").cpu())
    assert torch.equal(wl.make_prompts(wl.LLADA_8B, "cpu", batch=4), wl.make_prompts(wl.LLADA_8B, "cuda", batch=4).cpu())
