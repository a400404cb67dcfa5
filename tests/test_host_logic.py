"""Host-side logic that needs no GPU: shape tables, counts, the input generator."""
import numpy as np
import torch

from paper_2609_28568_b200 import shapes, synth


def _golden_counts(golden_dir):
    d = {}
    for line in open(f"{golden_dir}/model_counts.txt"):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        d[k] = int(v)
    return d


def test_parameter_counts_match_paper(golden_dir):
    g = _golden_counts(golden_dir)
    n, t = shapes.gpt2_param_count()
    assert n == g["gpt2_124m_parameters"]
    assert t == g["gpt2_124m_tensors"]
    assert shapes.qwen3_lora_param_count(16) == g["qwen3_lora_r16_parameters"]
    assert 3 * 19 * 1024 * 9 == g["tokens_per_step_run"]
    assert 16 * 1024 * 16 == g["tokens_per_step_speed"]


def test_flop_accounting():
    assert shapes.gpt2_stack_flops_per_token() == 741408768
    assert shapes.qwen3_stack_flops_per_token(True) == 2642411520
    assert shapes.qwen3_stack_flops_per_token(False) * 3 == shapes.qwen3_stack_flops_per_token(True) * 2
    blk = shapes.gpt2_block()
    assert [s.OC for s in blk] == [2304, 768, 3072, 768]
    assert shapes.VOCAB_PADDED % 128 == 0 and shapes.VOCAB_PADDED - shapes.VOCAB_REAL == 47


def test_synth_is_reproducible_and_addressable():
    a = synth.normal(1234, (37, 24), 0.02)
    b = synth.normal(1234, (37, 24), 0.02)
    assert a.dtype == torch.bfloat16 and torch.equal(a, b)
    rows = [0, 5, 36]
    assert torch.equal(synth.normal_rows(1234, rows, 24, 0.02), a[rows])
    assert torch.equal(synth.normal_flat(1234, 24 * 5, 24, 0.02), a[5])
    assert not torch.equal(synth.normal(1235, (37, 24), 0.02), a)
    # indices above 2^32 hash differently from their low words
    hi = synth.normal_flat(7, (1 << 32) + 3, 8, 1.0)
    lo = synth.normal_flat(7, 3, 8, 1.0)
    assert not torch.equal(hi, lo)


def test_synth_distribution():
    x = synth.normal(99, (1 << 18,), 1.0).float().numpy()
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01
    assert abs(np.mean(np.abs(x) < 1.0) - 0.6827) < 0.01
    y = synth.normal(100, (1 << 16,), 1e-3).float().numpy()
    assert abs(y.std() - 1e-3) < 2e-5
    # neighbouring elements are uncorrelated
    assert abs(np.corrcoef(x[:-1], x[1:])[0, 1]) < 0.01


def test_vocab_padding_helpers():
    w = synth.normal(5, (synth.VOCAB_PADDED, 8), 0.02)
    synth.zero_pad_vocab_rows(w)
    assert torch.all(w[synth.VOCAB_REAL:] == 0) and torch.any(w[:synth.VOCAB_REAL] != 0)
    d = synth.normal(6, (4, synth.VOCAB_PADDED), 1e-4)
    synth.zero_pad_vocab_cols(d)
    assert torch.all(d[:, synth.VOCAB_REAL:] == 0)


def test_tensor_seed_formula():
    assert synth.tensor_seed(4, 11, 3, 2) == 1337 + 4000 + 1100 + 30 + 2
