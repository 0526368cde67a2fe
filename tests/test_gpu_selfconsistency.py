"""Seeded random shapes through the prefill: a repeated call gives the same bits, and the rows from a random
cut n0 on, computed as appended rows, are bit-identical to the single shot (tile-aligned cuts when the inputs are
the outlier variant: see atf_prefill_chunk for the one rounding-sized exception).  No oracle here: this checks the
kernel's indexing (ragged tails, offsets, short and long walks, both head sizes, GQA ratios) against itself."""
import random

import pytest
import torch

import atf_inputs as gen

pytestmark = pytest.mark.gpu


def test_random_shapes_repeat_and_chunk_bit_identical():
    import paper_2608_02947_b200 as atf
    atf.lib()
    rnd = random.Random(7)
    for case in range(60):
        d = rnd.choice([64, 128]); B = rnd.choice([1, 2]); Hkv = rnd.choice([1, 2]); Hq = Hkv * rnd.choice([1, 2, 3])
        N = rnd.choice([1, 2, 127, 128, 129, 255, 256, 257, 383, 500, 777, 1024, 1500, 2049, 3000])
        k = rnd.choice([0.5, 2.0, 8.0, float("inf")]); base = rnd.choice([1e4, 1e6]); mode = rnd.choice([0, 1])
        outlier = rnd.random() < 0.2
        w = gen.Workload("s", B, Hq, Hkv, d, N, base, k, None, gen.SEED0 + 1000 + case, outlier)
        W, theta = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
        Q, K, V = gen.prefill_inputs(w, device="cuda")
        atf.atf_rope(Q, theta)
        atf.atf_rope(K, theta)
        O, L = atf.atf_prefill(Q, K, V, table=W, mode=mode)
        O2, L2 = atf.atf_prefill(Q, K, V, table=W, mode=mode)
        tag = (case, d, B, Hq, Hkv, N, k, base, mode, outlier)
        assert torch.isfinite(L).all(), tag
        assert torch.equal(O, O2) and torch.equal(L, L2), tag
        if N > 1:
            n0 = rnd.randrange(1, N)
            if outlier:
                n0 = max(128, n0 // 128 * 128) if N > 128 else 0
            if 0 < n0 < N:
                Oc, Lc = atf.atf_prefill(Q[:, :, n0:].contiguous(), K, V, table=W, mode=mode)
                assert torch.equal(Oc, O[:, :, n0:]) and torch.equal(Lc, L[:, :, n0:]), tag + (n0,)
    torch.cuda.synchronize()
    atf.binding.check_status()
