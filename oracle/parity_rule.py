"""How a result is compared with the oracle's (TEST INFRASTRUCTURE, like the rest of oracle/).

Used by the GPU parity tests and by the benchmark's CPU-baseline leg, which checks the timed run's bounds
against the oracle boxes it computes anyway.  Nothing here computes bounds; it only compares arrays.

Tolerance: |x - oracle| <= TOL * (1 + |oracle|) per bound.  Branch codes (Relu transformer of the DeepPoly
listing, Appendix C) must be identical wherever float32 can reproduce the decision: the oracle reports, per
ReLU neuron, margin = min(|l|, |u|, |l + u|) / (1 + max(|l|, |u|)); a neuron below MARGIN_MIN is a near-tie
whose sign tests float32 rounding may flip.
"""
import numpy as np

TOL = 1e-4
MARGIN_MIN = 1e-5


def layer_layout(layers):
    """Per affine layer: (offset in a bounds row, neurons, offset in a branch-code row or -1 without a ReLU)."""
    out, off, roff = [], 0, 0
    for l in layers:
        n = l.n_out
        out.append((off, n, roff if l.relu_after else -1))
        off += n
        if l.relu_after:
            roff += n
    return out


def comparable_prefix(codes, ref_codes, margins, layout):
    """Which affine layers of one box can be held to the tolerance.

    The bounds of layer k depend on the relaxations of the ReLU layers below it only.  A neuron whose sign
    tests are all at least MARGIN_MIN from zero must get the oracle's branch code; a near-tie may
    legitimately get either, and when it does get the other one the relaxation used above it differs, so the
    layers above are not compared for this box.  Everything up to and including the layer of that neuron is:
    its bounds were computed before its relaxation was chosen.
    Returns (number of leading layers to compare, mask of codes that must match, near-tie neurons seen)."""
    mask = np.zeros(ref_codes.shape, dtype=bool)
    ties = 0
    for k, (_, n, roff) in enumerate(layout):
        if roff < 0:
            continue
        firm = margins[roff:roff + n] >= MARGIN_MIN
        mask[roff:roff + n] = firm
        ties += int((~firm).sum())
        if (codes[roff:roff + n][~firm] != ref_codes[roff:roff + n][~firm]).any():
            return k + 1, mask, ties
    return len(layout), mask, ties


def parity_report(lb, ub, codes, ref, layers):
    """Compares bounds lb, ub [boxes, n_total] and codes [boxes, n_relu] with the oracle result `ref` of the same
    boxes under the rule above.  Returns counts and the worst scaled error; asserts nothing."""
    layout = layer_layout(layers)
    n_boxes = lb.shape[0]
    worst, mismatches, ties, pairs, cut, neurons = 0.0, 0, 0, 0, 0, 0
    for b in range(n_boxes):
        n_layers, mask, t = comparable_prefix(codes[b], ref["codes"][b], ref["margins"][b], layout)
        ties += t
        pairs += n_layers
        cut += n_layers < len(layout)
        end = layout[n_layers - 1][0] + layout[n_layers - 1][1]
        neurons += end
        for g, r in ((lb[b, :end], ref["lb"][b, :end]), (ub[b, :end], ref["ub"][b, :end])):
            worst = max(worst, float((np.abs(g - r) / (1.0 + np.abs(r))).max(initial=0.0)))
        rend = 0
        for (_, n, roff) in layout[:n_layers]:
            if roff >= 0:
                rend = roff + n
        m = mask[:rend]
        mismatches += int((codes[b, :rend][m] != ref["codes"][b, :rend][m]).sum())
    margins = ref["margins"]
    return {"boxes": int(n_boxes), "boxes_cut_short": int(cut), "layer_pairs_compared": int(pairs),
            "share_compared": round(pairs / float(max(1, n_boxes * len(layout))), 4),
            "bounds_compared": int(2 * neurons), "near_ties": int(ties), "code_mismatches": int(mismatches),
            "max_scaled_err": float(worst), "min_margin": float(margins.min()) if margins.size else None}
