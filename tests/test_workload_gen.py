"""The seeded input generators: hashing, dtype conversion, shapes and distributions (no GPU)."""
import numpy as np
import torch
from scipy import stats

from paper_2602_10273_b200.workload import gen as W


def test_hash_matches_scalar_definition():
    def sm(x):
        z = (x + 0x9E3779B97F4A7C15) % 2**64
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) % 2**64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) % 2**64
        return z ^ (z >> 31)

    want = sm(sm(sm(sm(sm(3) ^ 4) ^ 5) ^ 6) ^ 7)
    assert int(W.hash5(3, 4, 5, 6, 7)) == want
    arr = W.hash5(3, 4, np.array([5, 9]), 6, np.array([[7], [8]]))
    assert arr.shape == (2, 2) and int(arr[0, 0]) == want


def test_bf16_conversion_agrees_with_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 10, 5000), [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38, -1e-40]]).astype(np.float32)
    bits = W.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    back = W.bf16_bits_to_f32(bits)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_vocab_bias_is_a_zipf_profile_over_a_permutation():
    V = 1000
    b = W.vocab_bias(5, V, 1.5)
    assert np.allclose(np.sort(b)[::-1], -1.5 * np.log1p(np.arange(V)))
    assert not np.array_equal(np.argsort(-b), np.arange(V))
    assert not np.array_equal(W.vocab_bias(6, V, 1.5), b)


def test_logits_block_is_first_order_and_gaussian():
    V = 4096
    bias = np.zeros(V)
    a = W.logits_block(1, 3, [0, 0, 1], [10, 10, 10], V, 2.0, bias, "f32")
    assert a.shape == (3, V) and a.dtype == np.float32
    assert np.array_equal(a[0], a[1]) and not np.array_equal(a[0], a[2])       # same (group, t, prev) => same row
    b = W.logits_block(1, 4, [0], [10], V, 2.0, bias, "f32")
    c = W.logits_block(1, 3, [0], [11], V, 2.0, bias, "f32")
    assert not np.array_equal(a[0], b[0]) and not np.array_equal(a[0], c[0])
    assert stats.kstest(a[0] / 2.0, "norm").pvalue > 1e-3
    h = W.logits_block(1, 3, [0], [10], V, 2.0, bias, "bf16")
    assert h.dtype == np.uint16 and np.array_equal(h[0], W.f32_to_bf16_bits(a[0]))
    with_bias = W.logits_block(1, 3, [0], [10], V, 2.0, W.vocab_bias(1, V, 1.5), "f32")
    assert np.allclose(with_bias[0] - a[0], W.vocab_bias(1, V, 1.5), atol=1e-5)


def test_kv_block_rows_are_distinct():
    k = W.kv_block(2, 1, 0, [0, 1, 5], 2, 8, 16, "f32")
    v = W.kv_block(2, 1, 1, [0, 1, 5], 2, 8, 16, "f32")
    assert k.shape == (3, 2, 8, 16)
    flat = k.reshape(3 * 2 * 8, 16)
    assert len({r.tobytes() for r in flat}) == flat.shape[0]
    assert not np.array_equal(k, v)
    assert np.array_equal(W.kv_block(2, 1, 0, [5], 2, 8, 16, "f32")[0], k[2])
    assert stats.kstest(W.kv_block(2, 0, 0, [0], 4, 64, 64, "f32").ravel(), "norm").pvalue > 1e-3


def test_prompt_helpers_and_config_table():
    pl = W.prompt_lengths(1, 64, 64, 256)
    assert pl.min() >= 64 and pl.max() <= 256 and len(set(pl.tolist())) > 20
    assert np.array_equal(W.prompt_lengths(1, 4, 512, 512), [512] * 4)
    lt = W.prompt_last_token(1, 64, pl, 128256)
    assert lt.min() >= 0 and lt.max() < 128256
    c = W.CONFIGS
    assert [c[k].R for k in ("tiny", "llama2_7b", "qwen25_7b", "resample_stress", "batched_prompts")] == [4, 8, 16, 32, 512]
    assert c["tiny"].kv_bytes_per_pos_per_row == 2048 and c["llama2_7b"].kv_bytes_per_pos_per_row == 524288
    assert c["qwen25_7b"].kv_bytes_per_pos_per_row == 57344 and c["batched_prompts"].kv_bytes_per_pos_per_row == 131072
    assert c["batched_prompts"].logit_bytes_per_row == 256512 and c["resample_stress"].logit_bytes_per_row == 303872
    for w in c.values():
        assert w.max_len >= w.prompt_hi + w.T and w.eos_id == w.V - 1 and abs(w.tau * w.alpha - 1.0) < 1e-12
