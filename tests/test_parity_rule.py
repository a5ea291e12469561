"""The rule the GPU parity tests use for near-tie neurons, checked on the CPU with the oracle playing both
parts: a planted difference must be caught where the rule says it is compared, and only there."""
import numpy as np
import pytest

from oracle import deeppoly_oracle as orc
from paper_2507_20055_b200 import workloads as wl
from parity_util import MARGIN_MIN, compare, comparable_prefix, layer_layout


def _case():
    w = wl.small_fc([12, 20, 20, 20, 4], batch=3, eps=0.05, seed=11)
    ref = orc.deeppoly(w.layers, w.centers, w.eps, w.clip_lo, w.clip_hi)
    gpu = {"lb": ref["lb"].astype(np.float32), "ub": ref["ub"].astype(np.float32), "codes": ref["codes"].copy(),
           "status": 0, "layers": w.layers}
    ref = {k: v.copy() for k, v in ref.items()}
    ref["margins"] = np.maximum(ref["margins"], 10 * MARGIN_MIN)      # every neuron firm unless a test says otherwise
    return w, gpu, ref


def test_identical_results_compare_everything():
    w, gpu, ref = _case()
    r = compare(gpu, ref, label="same")
    assert r["layer_pairs_compared"] == w.batch * len(w.layers) and r["boxes_cut_short"] == 0


def test_a_firm_neuron_with_another_code_fails():
    w, gpu, ref = _case()
    gpu["codes"][1, 25] ^= 1
    with pytest.raises(AssertionError, match="branch codes differ"):
        compare(gpu, ref, label="firm flip")


def test_a_near_tie_resolved_differently_cuts_the_box_above_that_layer_only():
    w, gpu, ref = _case()
    # neuron 5 of the second ReLU layer (offset 20) of box 1 is a near-tie and the GPU picked the other slope
    ref["margins"][1, 25] = 0.1 * MARGIN_MIN
    gpu["codes"][1, 25] ^= 1
    gpu["lb"][1, 40:] += 1.0          # everything above layer 2 may differ for this box ...
    r = compare(gpu, ref, label="tie flip")
    assert r["boxes_cut_short"] == 1 and r["layer_pairs_compared"] == w.batch * len(w.layers) - 2
    gpu["lb"][1, 39] += 1.0           # ... but layer 2's own bounds were computed before the tie mattered
    with pytest.raises(AssertionError, match="scaled error"):
        compare(gpu, ref, label="tie flip, wrong bound below")


def test_a_near_tie_resolved_alike_keeps_the_whole_box():
    w, gpu, ref = _case()
    ref["margins"][0, 3] = 0.0
    r = compare(gpu, ref, label="tie, same code")
    assert r["boxes_cut_short"] == 0 and r["near_ties"] == 1
    gpu["ub"][0, -1] += 1.0
    with pytest.raises(AssertionError, match="scaled error"):
        compare(gpu, ref, label="tie, same code, wrong bound above")


def test_firm_neurons_beside_a_tie_are_still_held_to_their_codes():
    w, gpu, ref = _case()
    ref["margins"][2, 7] = 0.0
    gpu["codes"][2, 7] ^= 1           # allowed
    gpu["codes"][2, 9] ^= 1           # same layer, firm: not allowed
    with pytest.raises(AssertionError, match="branch codes differ"):
        compare(gpu, ref, label="firm beside tie")


def test_too_little_left_to_compare_fails():
    w, gpu, ref = _case()
    ref["margins"][:, 0] = 0.0
    gpu["codes"][:, 0] ^= 1           # every box cut after the first layer
    with pytest.raises(AssertionError, match="could be compared"):
        compare(gpu, ref, label="all cut")


def test_prefix_of_a_net_with_a_layer_without_relu():
    w = wl.small_fc([6, 8, 8, 8, 3], batch=1, eps=0.1, seed=12)
    w.layers[1].relu_after = False
    layout = layer_layout(w.layers)
    assert [x[2] for x in layout] == [0, -1, 8, -1]
    codes = np.zeros(16, np.uint8)
    margins = np.ones(16)
    margins[9] = 0.0
    other = codes.copy()
    other[9] = 2
    n, mask, ties = comparable_prefix(other, codes, margins, layout)
    assert n == 3 and ties == 1 and mask.sum() == 15
