"""Where may two runs of the greedy round part?  Only at a decision the oracle itself takes by a margin
inside the error of its inputs.

The round is a chain of comparisons between gains (w v' - w v) / units built from curve values.  Two
chains that read curve values differing by at most `tol` relative (single- against double-precision
tables, or single- against double-precision arithmetic on one table) must take the same decisions until
the first one whose margin, in the oracle's own numbers, is within what such a perturbation can move:
    gain_a - gain_b <= err_a + err_b,   err = (tol + ARITH) * w * (v' + v) / units
(ARITH covers the single-precision roundings of the gain's own three operations), or an accept / reject
test v' > v whose two values are within tol of each other, or a curve entry that the two tables resolve
to different plans or GPU counts (plans of equal predicted throughput).  No arithmetic of the method
lives here: the numbers come from the oracle's candidate dump.
"""
import numpy as np

ARITH = 2.5e-7


def decode(entry):
    """step-log entry -> (job, type, accepted)"""
    return int(entry) >> 2, (int(entry) >> 1) & 1, int(entry) & 1


def first_difference(log_a, log_b):
    """Index of the first entry in which two step logs differ; the shorter length when one is a proper
    prefix of the other; None when they are equal."""
    n = min(len(log_a), len(log_b))
    diff = np.nonzero(np.asarray(log_a[:n]) != np.asarray(log_b[:n]))[0]
    if len(diff):
        return int(diff[0])
    return None if len(log_a) == len(log_b) else n


def oracle_pick(cand):
    """The decision the round's rule takes from a candidate dump: largest positive GPU gain among offers that
    can be placed, else largest positive CPU gain, lowest job on ties.  -> (job, type) or None."""
    for t in (0, 1):
        ok = (cand["shut"][:, t] == 0) & (cand["next"][:, t] >= 0) & (cand["placeable"][:, t] != 0) & (cand["gain"][:, t] > 0)
        if ok.any():
            return int(np.argmax(np.where(ok, cand["gain"][:, t], -np.inf))), t
    return None


def assert_divergence_is_a_near_tie(run_oracle, log_o, log_x, w, tol, entries_differ=None):
    """run_oracle(k) -> the oracle's round stopped before step k, with its candidate dump (`cand`);
    log_o / log_x: step logs of the oracle and of the other chain; w [J] job weights; tol: largest relative
    difference between the curve values the two chains read.  entries_differ(job, g level, c level, m level)
    -> bool (optional): do the two chains' tables hold another plan or GPU count at that curve entry?
    Returns None when the logs agree, else a short description of the near tie at the first difference;
    raises AssertionError when the first difference is not a near tie."""
    k = first_difference(log_o, log_x)
    if k is None:
        return None
    r = run_oracle(k)
    cand = r["cand"]
    assert r["steps"] == k
    mine = oracle_pick(cand)
    assert mine == (decode(log_o[k])[:2] if k < len(log_o) else None), "the candidate dump does not reproduce the oracle's own decision"
    w = np.asarray(w, dtype=np.float64)
    err = (tol + ARITH) * w[:, None] * (cand["v_next"] + cand["v_cur"]) / np.maximum(cand["units"], 1.0)
    live = (cand["shut"] == 0) & (cand["next"] >= 0) & (cand["placeable"] != 0)
    theirs = decode(log_x[k]) if k < len(log_x) else None

    if theirs is None:
        clear = live & (cand["gain"] > err)
        assert not clear.any(), f"step {k}: the other chain stopped while the oracle had a clear gain left"
        return f"step {k}: the other chain stopped; the oracle's remaining gains are within rounding of zero"
    jx, tx, okx = theirs
    if mine is None:
        # the oracle saw no positive gain; the other chain's increment must be one whose two values nearly coincide
        assert cand["shut"][jx, tx] == 0, f"step {k}: the other chain moved job {jx}, which the oracle has shut out"
        assert abs(cand["gain"][jx, tx]) <= max(err[jx, tx], (tol + ARITH) * w[jx] * 2 * cand["v_cur"][jx, tx]), \
            f"step {k}: the other chain went on where the oracle saw no gain"
        return f"step {k}: the oracle stopped; the other chain's gain is within rounding of zero"
    jo, to = mine
    if (jo, to) == (jx, tx):
        # same increment, accepted by one chain only: the test v' > v at the commit level, or an entry the tables resolve differently
        vc, vcur = cand["v_commit"][jo, to], cand["v_cur"][jo, to]
        close = abs(vc - vcur) <= (tol + ARITH) * max(vc, vcur)
        other = entries_differ is not None and cand["m_commit"][jo, to] >= 0 and entries_differ(
            jo, int(cand["gi"][jo, to]), int(cand["ci"][jo, to]), int(cand["m_commit"][jo, to]))
        assert close or other, f"step {k}: job {jo} accepted by one chain only, with values {vc!r} against {vcur!r}"
        return f"step {k}: increment of job {jo} accepted by one chain only; deciding values within {tol + ARITH:.2g}"
    if to != tx:
        # GPU increments come first: one chain still saw one where the other had none left
        jg, tg = (jo, to) if to == 0 else (jx, tx)
        assert cand["gain"][jg, tg] <= err[jg, tg], f"step {k}: a clear GPU gain of job {jg} was seen by one chain only"
        return f"step {k}: GPU gain of job {jg} within rounding of zero"
    assert live[jx, tx], f"step {k}: the other chain picked job {jx}, which the oracle cannot place or has shut out"
    gap = cand["gain"][jo, to] - cand["gain"][jx, tx]
    bound = err[jo, to] + err[jx, tx]
    assert gap <= bound, (f"step {k}: the oracle prefers job {jo} (gain {cand['gain'][jo, to]!r}) to job {jx} "
                          f"(gain {cand['gain'][jx, tx]!r}) by more than rounding allows ({bound!r})")
    return f"step {k}: gains of jobs {jo} and {jx} differ by {gap:.3g}, within {bound:.3g}"
