"""Pins for the oracle's search procedures, recomputed step by step in numpy from the oracle's primitive
operations (quantise, table statistics, refit) instead of trusting its drivers:

* Algorithm 1 as printed (no rate correction afterwards): the twelve geometric bisections of the scale on the
  fixed row sample, the full-tensor fit test, precision escalation;
* its last resort at the highest precision (App. "Scale-search settings"): s <- 1.05 s A_max / 2^b until the
  alphabets fit;
* Alg. 2 (Sec. 3.5) on a case small enough to enumerate: Eq. 14 under the half-count-smoothed shared model, the
  budget of Eq. 15, and the common rate penalty of Eq. 16.

The library's host encoder must give the oracle's bytes in every case."""
import itertools

import numpy as np

import oracle
import paper_2609_34185_b200 as ep
from paper_2609_34185_b200 import synth


def _bisect_scale(W, target, b, V, rows, steps=12, lo=1e-3, hi=8.0, retained=16.0):
    """Algorithm 1's inner loop on the row sample: returns the fp32 scale after `steps` bisections."""
    Ws = np.ascontiguousarray(W[rows])
    for _ in range(steps):
        s = np.sqrt(lo * hi)
        fields, _ = oracle.quantise(Ws, float(np.float32(s)))
        st = oracle.model_stats(fields, rows=len(rows), b=b, V=V, retained=retained)
        if st["observed"].max() > (1 << b):          # no b-bit table exists for this sample: too fine a scale
            lo = s
            continue
        rate = st["est_bits"] / Ws.size              # Eq. 12: 8 B_sub / N_sub
        if rate > target:
            lo = s
        else:
            hi = s
    return np.float32(np.sqrt(lo * hi))


def _fit(W, s, b, V):
    fields, _ = oracle.quantise(W, float(s))
    obs = oracle.model_stats(fields, rows=W.shape[0], b=b, V=V)["observed"]
    return int(obs.max()), int(obs[1:].max())


def test_algorithm_1_as_printed_step_by_step():
    for W, target, budget in ((synth.student_t_rows(192, 1024, 41), 3.0, 1 << 13),
                              (synth.gaussian_rows(64, 2048, 42), 5.0, 1 << 18),
                              (synth.laplace_rows(128, 512, 43), 2.0, 1 << 12)):
        R, C = W.shape
        V = oracle.default_tile_vectors(target)
        rows = oracle.sample_rows(R, C, budget)
        opts = oracle.default_opts(polish_steps=0, sample_vectors=budget)
        blob, rep = oracle.encode(W, target, opts)
        b = 11
        while True:                                  # precision escalation: raise b until the full tensor fits
            s = _bisect_scale(W, target, b, V, rows)
            worst, _ = _fit(W, s, b, V)
            if worst <= (1 << b):
                break
            b += 1
        assert rep["b"] == b and np.float32(rep["s"]) == s, (rep["s"], float(s), rep["b"], b)
        assert rep["sample_rows"] == len(rows)
        lib = ep.encode(W, target, polish_steps=0, sample_vectors=budget)
        assert np.array_equal(lib.data, blob)
        # the printed procedure alone lands within a few percent of the target (small row samples here)
        assert abs(rep["stored_bpp"] - target) < 0.06 * target


def test_coarsening_at_the_highest_precision():
    # the sampled rows are uniformly distributed (few distinct coordinates), all other rows Laplacian: the scale
    # found on the sample at 9 bpp gives the full tensor more than 2^9 symbols per coordinate table, and with b
    # already at its maximum the scale grows by 1.05 A_max / 2^b per round until the alphabets fit
    R, C, b, target, budget = 128, 4096, 9, 9.0, 1 << 13
    rows = oracle.sample_rows(R, C, budget)
    assert len(rows) == 16
    rng = np.random.Generator(np.random.PCG64(45))
    W = synth.laplace_rows(R, C, 44)
    W[rows] = rng.uniform(-0.02, 0.02, (len(rows), C)).astype(np.float32)
    V = oracle.default_tile_vectors(target)
    opts = oracle.default_opts(polish_steps=0, sample_vectors=budget, b_start=b, b_max=b)
    blob, rep = oracle.encode(W, target, opts)
    s = _bisect_scale(W, target, b, V, rows)
    s0, rounds = s, 0
    while True:
        worst, amax = _fit(W, s, b, V)
        if worst <= (1 << b):
            break
        s = np.float32(1.05 * float(s) * amax / (1 << b))
        rounds += 1
        assert rounds < 50
    assert rounds >= 1 and s > s0                    # the branch was taken
    assert rep["b"] == b and np.float32(rep["s"]) == s, (rep["s"], float(s), rounds)
    info = oracle.info(blob)
    assert info["b"] == b
    lib = ep.encode(W, target, polish_steps=0, sample_vectors=budget, b_start=b, b_max=b)
    assert np.array_equal(lib.data, blob)
    # with the rate correction on top the two encoders still agree
    assert np.array_equal(ep.encode(W, target, sample_vectors=budget, b_start=b, b_max=b).data,
                          oracle.encode(W, target, oracle.default_opts(sample_vectors=budget, b_start=b, b_max=b))[0])


# ---- Alg. 2 on a case small enough to enumerate ------------------------------------------------------

def _table_ids(fields):
    """table of every symbol of every block: 0 for the coset, 1 + 8c + (k - 1) for field k under coset c"""
    c = fields[:, 0]
    t = np.zeros(fields.shape, np.int64)
    t[:, 1:] = 1 + 8 * c[:, None] + np.arange(8)[None, :]
    return t


def _points(fields):
    c = fields[:, 0].astype(np.float64)
    p = np.empty((len(fields), 8))
    p[:, :7] = fields[:, 1:8] + 0.5 * c[:, None]
    p[:, 7] = 2 * fields[:, 8] + (fields[:, 1:8].sum(axis=1) % 2) + 0.5 * c
    return p


def test_per_row_refinement_on_an_enumerable_case():
    R, C, K, target = 4, 512, 3, 3.0
    W = synth.gaussian_rows(R, C, 46, lo=0.01, hi=0.02)
    W[1] *= np.float32(1.0) + 0.5 * np.sin(np.arange(C, dtype=np.float32))      # rows that favour different ratios
    W[3, ::7] *= np.float32(4.0)
    per_row = C // 8
    base_blob, base = oracle.encode(W, target)
    s, b, V = np.float32(base["s"]), base["b"], base["V"]
    rho = oracle.rdo_ratios(K)
    cand, sig, D = [], [], np.zeros((R, K))
    mu = None
    for k in range(K):
        sk = np.float32(rho[k] * float(s))
        f, mu = oracle.quantise(W, float(sk))
        g = oracle.refit(W, f, float(sk), mu)
        cand.append(f.reshape(R, per_row, 9))
        sig.append(g)
        P = _points(f).reshape(R, C)
        D[:, k] = ((W.astype(np.float64) - g.astype(np.float64)[:, None] * P) ** 2).sum(axis=1)
    # Eq. 14 under the shared model of the current (baseline) selection: counts plus one half over the value
    # range all candidates span, per table
    allf = np.concatenate([c.reshape(-1, 9) for c in cand])
    allt = _table_ids(allf)
    f0 = cand[0].reshape(-1, 9)
    t0 = _table_ids(f0)
    nl = {}
    for t in np.unique(allt):
        lo, hi = allf[allt == t].min(), allf[allt == t].max()
        w = hi - lo + 1
        cnt = np.bincount(f0[t0 == t] - lo, minlength=w).astype(np.float64)
        nl[t] = (lo, -np.log2((cnt + 0.5) / (cnt.sum() + 0.5 * w)))
    Rr = np.zeros((R, K))
    for k in range(K):
        for r in range(R):
            f = cand[k][r]
            t = _table_ids(f)
            Rr[r, k] = sum(nl[tt][1][v - nl[tt][0]] for tt, v in zip(t.reshape(-1), f.reshape(-1)))
    budget = Rr[:, 0].sum()                          # Eq. 15 with one sweep: mixture = baseline, B = B_mix
    # what the oracle chose: read the refined stream back and match each row's fields with a candidate
    blob, _ = oracle.encode(W, target, oracle.default_opts(rdo_candidates=K, rdo_sweeps=1))
    _, got = oracle.decode(blob, oracle.FP32, want_fields=True)
    got = got.reshape(R, per_row, 9)
    chosen = []
    for r in range(R):
        ks = [k for k in range(K) if np.array_equal(got[r], cand[k][r])]
        assert ks, r
        chosen.append(ks[0])
    scales = np.frombuffer(blob[oracle.info(blob)["off_scales"]:][:4 * R].tobytes(), np.float32)
    assert all(scales[r] == sig[chosen[r]][r] for r in range(R))          # the candidate's own refitted scale
    rate = lambda sel: sum(Rr[r, k] for r, k in enumerate(sel))
    dist = lambda sel: sum(D[r, k] for r, k in enumerate(sel))
    assert rate(chosen) <= budget + 1e-9
    assert dist(chosen) <= dist([0] * R) + 1e-18
    # Eq. 16: kappa_lambda(r) = argmin_k D + lambda R (lowest k on ties); over a fine grid of penalties no selection
    # inside the budget has lower distortion than the oracle's
    best = None
    for lam in np.concatenate([[0.0], np.geomspace(1e-12, 1e3, 6000) * D.sum() / Rr.sum()]):
        sel = [int(np.argmin(D[r] + lam * Rr[r])) for r in range(R)]
        if rate(sel) <= budget and (best is None or dist(sel) < best):
            best = dist(sel)
    assert best is not None and dist(chosen) <= best * (1 + 1e-12)
    # all 81 selections: the unconstrained optimum inside the budget bounds what any common penalty can reach
    exhaustive = min(dist(sel) for sel in itertools.product(range(K), repeat=R) if rate(sel) <= budget)
    assert exhaustive <= dist(chosen) * (1 + 1e-12)
    assert dist(chosen) <= 1.05 * exhaustive           # and the Lagrangian search gets close to it here
    assert len(set(chosen)) > 1                        # rows really went different ways
    lib = ep.encode(W, target, rdo_candidates=K, rdo_sweeps=1)
    assert np.array_equal(lib.data, blob)
    assert np.array_equal(ep.encode(W, target).data, base_blob)
