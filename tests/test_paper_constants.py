"""The workload shapes and defaults agree with what the paper prints."""
import os

import oracle
from paper_2504_06323_b200 import workloads as wl


def golden():
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if len(line) == 2:
                out[line[0]] = float(line[1])
    return out


def test_shapes_match_the_papers_model_table():
    g = golden()
    c7, c8, c13 = wl.CONFIGS["llama7b"], wl.CONFIGS["llama3_8b"], wl.CONFIGS["llama2_13b"]
    assert len(wl.PROJECTIONS) == g["projections_per_layer"]
    assert (c7.n_layers, c7.hidden, c7.intermediate) == (g["llama7b_layers"], g["llama7b_attention_dim"], g["llama7b_ffn_dim"])
    assert c7.n_layers * len(wl.PROJECTIONS) == g["llama7b_pruning_targets"]
    assert (c8.n_layers, c8.intermediate) == (g["llama3_8b_layers"], g["llama3_8b_ffn_dim"])
    assert (c13.n_layers, c13.hidden, c13.intermediate) == (g["llama2_13b_layers"], g["llama2_13b_attention_dim"], g["llama2_13b_ffn_dim"])
    for c in (c7, c8, c13):
        assert c.tokens == g["calibration_samples"] * g["calibration_tokens_per_sample"]
        assert c.alpha >= g["alpha_min"]
    assert c7.shape("gate") == (11008, 4096) and c7.shape("down") == (4096, 11008)
    assert c8.shape("k") == (1024, 4096) and c8.shape("q") == (4096, 4096)


def test_allocation_spread_is_in_the_range_the_paper_reports():
    # Context only: at p = 0.8 the paper reports per-layer targets spanning 16.8 points and
    # per-projection targets spanning 30.1 points; the default spread 2*lambda lies between 0
    # and the larger of the two, and the reported asymmetric range contains p.
    g = golden()
    spread_proj = g["e2_projection_target_max"] - g["e2_projection_target_min"]
    assert 0 < 2 * wl.CONFIGS["llama7b"].lam <= spread_proj
    s, _, clamped = oracle.allocate_sparsity([1, 2, 9], [100] * 3, [4096] * 3, 3, 1, 0.8, spread_proj / 2)
    assert not clamped and s.min() < 0.8 < s.max() and abs((s.max() - s.min()) - spread_proj) < 1e-12
