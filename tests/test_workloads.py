"""The seeded input generators: shapes, determinism and the structure the configurations ask for
(outlier channels, spike units, Zipf-shaped expert loads).  No format arithmetic is involved."""
import numpy as np
import torch

import hif4_workloads as wl


def test_moe_routing_is_topk_of_a_zipf_popularity():
    r = wl.moe_routing()
    counts, off, tok = r["counts"].numpy(), r["offsets"].numpy(), r["token_of_row"].numpy()
    assert counts.sum() == wl.MOE_TOKENS * wl.MOE_TOPK and len(counts) == wl.MOE_EXPERTS
    assert np.array_equal(off, np.concatenate([[0], np.cumsum(counts)]))
    assert (np.bincount(tok, minlength=wl.MOE_TOKENS) == wl.MOE_TOPK).all(), "every token is routed to 8 experts"
    for g in range(wl.MOE_EXPERTS):                       # ... to 8 different ones
        rows = tok[off[g]:off[g + 1]]
        assert len(np.unique(rows)) == len(rows)
    # popularity ~ rank^-1.1: a few hot experts, a long tail of small ones, (almost) nobody empty
    assert 2500 < counts.max() < 4096 and 20 <= np.median(counts) <= 70 and (counts > 0).sum() >= 250
    r2 = wl.moe_routing()
    assert np.array_equal(r2["counts"].numpy(), counts), "seeded: same routing every time"
    assert not np.array_equal(wl.moe_routing(seed=7)["counts"].numpy(), counts)


def test_activation_generators_have_the_stated_structure():
    x, w = wl.single_layer()
    assert x.shape == (128, 512) and w.shape == (512, 512) and x.dtype == torch.bfloat16
    col_rms = x.float().pow(2).mean(0).sqrt()
    assert set(torch.topk(col_rms, 4).indices.tolist()) == {7, 130, 257, 500}
    assert abs(float(w.float().std()) - 0.02) < 0.002
    a = wl.llama_activations(64, 4096)
    col_rms = a.float().pow(2).mean(0).sqrt()
    assert int((col_rms > 10 * col_rms.median()).sum()) == 21          # ceil(0.5 % of 4096) channels x50
    assert torch.equal(a, wl.llama_activations(64, 4096))
    p = wl.prefill_activations(256, 512)
    row_rms = p.float().pow(2).mean(1).sqrt().log2()
    assert float(row_rms.min()) < -2.5 and float(row_rms.max()) > 2.5 and float(row_rms.min()) > -4.6 and float(row_rms.max()) < 4.6


def test_quantize_sweep_mix_and_spike_units():
    x = wl.quantize_sweep(2 ** 20).float()
    assert x.shape == (256, 4096)
    assert float(x[2::3].abs().max()) <= 1000.0 + 1e-3 and float(x[2::3].abs().median()) < 1.0    # uniform rows (spikes x1000 allowed)
    units = x.view(256, 64, 64)
    peak = units.abs().max(-1).values
    second = units.abs().topk(2, -1).values[..., 1]
    spike = (peak > 50 * second.clamp_min(1e-9)).float().mean()
    assert 0.003 < float(spike) < 0.03, "about 1 % of the units hold one spike"
