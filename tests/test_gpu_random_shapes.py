"""Seeded random shapes through the fused apply against the fp64 oracle: token counts,
slot counts, ranks, widths and adapter distributions drawn together, so that tile
shapes, lane shares and ragged tails meet in combinations the hand-picked cases miss."""
import numpy as np
import pytest
import torch

from paper_2605_13779_b200 import synth
import parity

pytestmark = pytest.mark.gpu


def _cases():
    rng = np.random.default_rng(20260513)
    out = []
    for it in range(24):
        T = int(rng.choice([1, 7, 33, 64, 257, 600, 1500]))
        S = int(rng.choice([1, 3, 8, 40, 130]))
        r_max = int(rng.choice([1, 8, 16, 32, 64]))
        ranks = np.minimum(rng.choice([1, 2, 5, 8, 16, 24, 32, 64], size=S), r_max).astype(np.int32)
        d = int(rng.choice([8, 72, 520, 1032, 2560, 4104]))
        n = int(rng.choice([8, 40, 264, 1024, 2184, 5128]))
        zipf = None if rng.random() < 0.5 else 1.1
        p_none = float(rng.choice([0.0, 0.1, 0.5]))
        out.append((it, T, S, r_max, ranks, d, n, zipf, p_none))
    return out


@pytest.mark.parametrize("spec", _cases(), ids=lambda s: f"{s[0]}-T{s[1]}-S{s[2]}-r{s[3]}-d{s[5]}-n{s[6]}")
def test_random_shape(spec):
    from paper_2605_13779_b200 import binding as mb, harness
    it, T, S, r_max, ranks, d, n, zipf, p_none = spec
    case = synth.random_dense_case(f"gpu/random/{it}", T=T, d=d, n=n, num_slots=S, ranks=ranks, r_max=r_max,
                                   p_none=p_none, zipf_s=zipf)
    dev = harness.upload_dense(case)
    plan = mb.mint_lora_plan(dev.table, dev.ids, dev.status)
    mb.mint_lora_apply_fused(dev.pool, dev.table, plan, dev.x, dev.y, dev.status)
    torch.cuda.synchronize()
    assert dev.status.cpu().numpy()[0] == 0
    y_ref, _, _ = parity.oracle_dense(case)
    y = harness.y_to_f64(dev.y)
    parity.assert_close(y, y_ref, case.name)
    none = case.ids < 0
    if none.any():
        np.testing.assert_array_equal(y[none], synth.bf16_bits_to_f64(case.y0)[none])
