"""Label construction and uniform-token-set statistics: the CUDA kernels against the oracle on seeded weights."""
import numpy as np
import pytest

import workloads as wl

pytestmark = pytest.mark.gpu


def _check(w, topk):
    import torch
    from oracle import adore_oracle as ao
    from paper_2407_02328_b200 import adore as lib
    L, B, H, S = w.shape
    half = topk // 2
    dw = torch.from_numpy(w).cuda()
    sets = torch.full((L, B, H, half), -7, dtype=torch.int32, device="cuda")
    count = torch.full((B, S), -7, dtype=torch.int32, device="cuda")
    label = torch.full((B, S), 9, dtype=torch.uint8, device="cuda")
    cov = torch.zeros((L, B), dtype=torch.float32, device="cuda")
    mass = torch.zeros((L, B), dtype=torch.float32, device="cuda")
    for _ in range(2):                               # a second call must not depend on what the first left behind
        lib.adore_label_tokens(dw, L, B, H, S, topk, torch.cuda.current_stream().cuda_stream, sets, count, label, cov, mass)
    torch.cuda.synchronize()
    o_sets, o_count, o_label, o_cov, o_mass = ao.attention_labels(w, topk)
    assert np.array_equal(sets.cpu().numpy(), o_sets)
    assert np.array_equal(count.cpu().numpy(), o_count)
    assert np.array_equal(label.cpu().numpy(), o_label)
    assert np.allclose(cov.cpu().numpy(), o_cov, rtol=0, atol=1e-6)
    assert np.allclose(mass.cpu().numpy(), o_mass, rtol=0, atol=1e-5)
    return o_label


def test_labels_small_and_ragged_shapes():
    _check(wl.slot_weights(31, 3, 2, 4, 41, nonzero=12, empty_frac=0.2), 12)
    _check(wl.slot_weights(32, 4, 3, 8, 513, nonzero=256, empty_frac=0.1), 256)
    _check(wl.slot_weights(33, 2, 2, 4, 1025, nonzero=512, empty_frac=0.05), 512)
    _check(wl.slot_weights(34, 2, 1, 3, 65, nonzero=5, empty_frac=0.0), 64)        # fewer positive weights than K/2


def test_labels_with_equal_weights_and_empty_rows():
    w = wl.slot_weights(35, 3, 2, 4, 97, nonzero=40, empty_frac=0.1)
    w = (np.ceil(w * 64) / 64).astype(np.float32)      # few distinct values: the lower slot must win among equals
    w[1, 0, 2] = 0.0                                   # a head with nothing kept
    w[:, 1] = 0.0                                      # a sequence with no weights at all
    lab = _check(w, 24)
    assert lab[1].sum() == 0


def test_labels_at_llama_shape_one_sequence():
    # 32 layers x 32 heads over a 1025-slot cache, K = 512: what config 4 emits for one sequence
    _check(wl.slot_weights(36, 32, 1, 32, 1025, nonzero=512, empty_frac=0.02), 512)


def test_labels_reject_too_many_slots():
    import torch
    from paper_2407_02328_b200 import adore as lib
    z = torch.zeros(8, device="cuda")
    with pytest.raises(lib.AdoreError) as e:
        lib.adore_label_tokens(z, 1, 1, 1, 5000, 8, 0, z, z, z, z, z)
    assert e.value.status == 8
