import numpy as np
import torch

import lsp_synth as S


def test_normal_matches_pure_python_restatement():
    x = S.normal((5, 7), seed=3, tensor_id=11, scale=1.0)
    flat = x.flatten().tolist()
    for i in [0, 1, 6, 7, 20, 34]:
        assert abs(flat[i] - S.normal_py(3, 11, i)) < 1e-6


def test_randint_matches_pure_python_restatement():
    x = S.randint((40,), seed=9, tensor_id=1000, high=2047).tolist()
    for i in [0, 3, 17, 39]:
        assert x[i] == S.randint_py(9, 1000, i, 2047)


def test_normal_moments_and_chunk_independence():
    x = S.normal((1 << 18,), 0, 5).double()
    assert abs(x.mean().item()) < 0.01
    assert abs(x.std().item() - 1.0) < 0.01
    assert x.abs().max().item() < 4.95
    # element i does not depend on how many elements are drawn
    y = S.normal((100,), 0, 5)
    assert torch.equal(y, S.normal((1 << 18,), 0, 5)[:100])


def test_bf16_rounding_is_last_step():
    a = S.normal((64,), 1, 2, 0.02, torch.bfloat16)
    b = S.normal((64,), 1, 2, 0.02, torch.float32).to(torch.bfloat16)
    assert torch.equal(a, b)


def test_prompt_avoids_mask():
    sh = S.config("cfg1").shape
    p = S.make_prompt(2, 500, sh, 0)
    assert p.min() >= 0 and p.max() < sh.vocab and (p != sh.mask_id).all()


def test_delimiter_bitmap_bits():
    bm = S.delimiter_bitmap(64, 1, 8).numpy()
    bits = np.unpackbits(bm, bitorder="little")
    assert bits[:10].tolist() == [0, 1, 1, 1, 1, 1, 1, 1, 1, 0]
