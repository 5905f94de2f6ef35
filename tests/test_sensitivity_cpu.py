"""The parity inputs must be able to expose a wrong kernel (CPU only, oracle only).

Each mutation below is a mistake a kernel could plausibly make (a parameter ignored, an operand shifted by one
column, blocks taken in the wrong order, the centring term dropped).  It is applied to the ORACLE's inputs, and the
oracle's result has to move by several times the regression bound the GPU parity tests assert on the same recipe and
shape; otherwise that recipe could not tell the mistake from rounding.  The "flat" recipe (parameters ~ N(0, 1/d), the
benchmark configurations) gives near-uniform softmaxes on which some of these mistakes are invisible, which is why the
parity tests also run the "peaked" and "structured" recipes; this file keeps them from drifting back.
"""
import numpy as np
import pytest

from oracle import kvcapsule_oracle as orc
from paper_2605_16439_b200 import workloads as wl

import kvc_testlib as tl


def _inputs(shape, p):
    T = p["T"]
    a = {k: tl.np64(p[k]) for k in ("q", "K_vis", "V_vis", "theta", "U", "mu")}
    a["K_txt"], a["V_txt"] = tl.np64(p["K_txt"])[:, :, :T], tl.np64(p["V_txt"])[:, :, :T]
    a["K_t"], a["V_t"] = orc.compress(a["K_vis"], a["V_vis"], p["idx"].numpy(), a["U"], a["mu"], shape.n)
    return a


def _decode(a, **over):
    b = dict(a, **over)
    return orc.decode_attend_fused(b["q"], b["K_t"], b["V_t"], b["theta"], b["U"], b["mu"], b["K_txt"], b["V_txt"])


MUTATIONS = {
    "theta ignored (all zeros)": lambda a: dict(theta=np.zeros_like(a["theta"])),
    "theta shifted by one column": lambda a: dict(theta=np.roll(a["theta"], 1, axis=2)),
    "theta shifted by one row": lambda a: dict(theta=np.roll(a["theta"], 1, axis=1)),
    "U shifted by one column": lambda a: dict(U=np.roll(a["U"], 1, axis=2)),
    "K_tilde blocks in reverse order": lambda a: dict(K_t=a["K_t"][:, :, ::-1]),
    "V_tilde blocks in reverse order": lambda a: dict(V_t=a["V_t"][:, :, ::-1]),
    "K_tilde rows shifted by one": lambda a: dict(K_t=np.roll(a["K_t"], 1, axis=3)),
    "text keys shifted by one row": lambda a: dict(K_txt=np.roll(a["K_txt"], 1, axis=2)),
    "text rows left out of the softmax": lambda a: dict(K_txt=a["K_txt"][:, :, :0], V_txt=a["V_txt"][:, :, :0]),
    "heads of a group swapped": lambda a: dict(q=a["q"][:, ::-1]),
}
# mutations that only matter where there is something to mix up
NEEDS_BLOCKS = ("K_tilde blocks in reverse order", "V_tilde blocks in reverse order")


@pytest.mark.parametrize("recipe", ["peaked", "structured"])
@pytest.mark.parametrize("ci,kw", tl.REDUCED_7B)
def test_every_mutation_moves_the_result_well_beyond_the_asserted_bound(ci, kw, recipe):
    shape = tl.small(wl.CONFIGS[ci], **kw)
    p = tl.make_problem(shape, wl.layer_seed(ci, 3), T=shape.T0 + 5, T_cap=shape.T0 + 64, recipe=recipe)
    a = _inputs(shape, p)
    ref = _decode(a)
    bound = tl.regression_bound(shape.dtype, float(np.abs(ref).max()))
    assert bound <= tl.TOL[shape.dtype]
    for name, mut in MUTATIONS.items():
        if name in NEEDS_BLOCKS and shape.R < 2:
            continue
        moved = float(np.abs(_decode(a, **mut(a)) - ref).max())
        assert moved >= 5.0 * bound, f"{name}: moves the output by {moved:.4f}, bound {bound:.4f}"


def test_mu_term_is_visible_on_the_structured_recipe():
    """Dropping (sum P) mu shifts every output channel by the vision probability mass times mu."""
    ci, kw = tl.REDUCED_7B[0]
    shape = tl.small(wl.CONFIGS[ci], **kw)
    p = tl.make_problem(shape, wl.layer_seed(ci, 3), T=shape.T0 + 5, T_cap=shape.T0 + 64, recipe="structured")
    a = _inputs(shape, p)
    ref = _decode(a)
    # the capsules stay as compressed with the true mu; only the decode side forgets the term
    moved = float(np.abs(_decode(a, mu=np.zeros_like(a["mu"])) - ref).max())
    assert moved >= 5.0 * tl.regression_bound(shape.dtype, float(np.abs(ref).max()))


def test_flat_recipe_is_insensitive_to_some_of_them():
    """Why the extra recipes exist: on N(0, 1/d) parameters a reversed block order hides inside the bf16 contract bound."""
    ci, kw = tl.REDUCED_7B[2]
    shape = tl.small(wl.CONFIGS[ci], **kw)
    p = tl.make_problem(shape, wl.layer_seed(ci, 3), T=shape.T0 + 5, T_cap=shape.T0 + 64, recipe="flat")
    a = _inputs(shape, p)
    ref = _decode(a)
    moved = float(np.abs(_decode(a, K_t=a["K_t"][:, :, ::-1]) - ref).max())
    assert moved < tl.TOL["bf16"]                                  # invisible to the contract bound alone ...
    assert moved > tl.regression_bound("bf16", float(np.abs(ref).max()))   # ... but not to the regression bound
