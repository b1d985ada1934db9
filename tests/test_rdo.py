"""Per-row rate-distortion refinement (Sec. 3.5, Alg. 2): candidate ratios against their closed form, the
library against the oracle byte for byte, and the effect the paper reports (lower weight error at the same
stored size)."""
import numpy as np
import pytest

import oracle
import paper_2609_34185_b200 as ep
from paper_2609_34185_b200 import synth


def test_candidate_ratios_are_nested_log_bisections_of_the_papers_range():
    r5 = oracle.rdo_ratios(5)
    # 1 first; then the wider half [1, 1.45] is bisected, then [0.70, 1], then the two quarters above 1
    want = [1.0, 1.45 ** 0.5, 0.70 ** 0.5, 1.45 ** 0.25, 1.45 ** 0.75]
    assert np.allclose(r5, want, rtol=1e-12)
    for K in (1, 2, 3, 8):
        assert np.array_equal(oracle.rdo_ratios(K), oracle.rdo_ratios(9)[:K])       # nested as K grows
    r = oracle.rdo_ratios(33)
    assert r.min() > 0.70 and r.max() < 1.45 and len(set(np.round(r, 12))) == 33


@pytest.mark.parametrize("maker,shape,bpp,K,T", [
    (synth.gaussian_rows, (128, 1024), 3.0, 5, 1),
    (synth.laplace_rows, (96, 512), 4.0, 3, 2),
    (synth.student_t_rows, (64, 512), 2.0, 7, 1),
])
def test_library_refinement_matches_oracle_and_lowers_the_error(maker, shape, bpp, K, T):
    W = maker(shape[0], shape[1], 77 + K)
    lib = ep.encode(W, bpp, rdo_candidates=K, rdo_sweeps=T)
    ora, _ = oracle.encode(W, bpp, oracle.default_opts(rdo_candidates=K, rdo_sweeps=T))
    assert np.array_equal(lib.data, ora)
    base = ep.encode(W, bpp)
    e0 = oracle.rel_l2(W, oracle.decode(base.data, oracle.FP32)[0])
    e1 = oracle.rel_l2(W, oracle.decode(lib.data, oracle.FP32)[0])
    assert e1 < e0                                           # the paper: 14.35 % -> 14.11 % at 3 bpp with K = 5, T = 1
    assert abs(lib.stored_bpp - base.stored_bpp) < 0.01 * bpp  # allocated under the baseline's storage budget
    assert ep.validate(lib.data) == 0


def test_one_candidate_or_no_sweep_is_the_baseline():
    W = synth.gaussian_rows(64, 512, 5)
    base = ep.encode(W, 4.0)
    assert np.array_equal(ep.encode(W, 4.0, rdo_candidates=1, rdo_sweeps=3).data, base.data)
    assert np.array_equal(ep.encode(W, 4.0, rdo_candidates=5, rdo_sweeps=0).data, base.data)
    assert np.array_equal(oracle.encode(W, 4.0, oracle.default_opts(rdo_candidates=4, rdo_sweeps=0))[0], base.data)
