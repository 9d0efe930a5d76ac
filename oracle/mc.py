"""Monte Carlo estimates of the two failure events.  TEST INFRASTRUCTURE ONLY.

Section 4, "Failure modes and budget allocation": the method fails when R < k
(insufficient recall) or R > M (buffer overflow), R being the rank of the
threshold.  Lemma 1 says the law of R depends on ranks only, so the simulation
needs no values: an input is a placement of the ranks 1..N on the positions
0..N-1.

`simulate_ranks` does the whole experiment on ranks: place the ranks, draw the
stratified sample of positions, take the t-th smallest sampled rank as R.
`failure_rate_exchangeable` covers large N, where a uniformly random placement
makes the number of sampled positions among any fixed set of ranks exactly
hypergeometric (whatever the sampling scheme, because the scheme does not look
at the ranks); the two events are disjoint, so their rates add.

These draws use NumPy's generator, not Philox: they estimate a law, they do not
reproduce the library's sample.
"""
from __future__ import annotations

import numpy as np


def stratified_positions(N: int, S: int, rng: np.random.Generator) -> np.ndarray:
    """One uniformly random position from each stratum [floor(jN/S), floor((j+1)N/S))."""
    b = (np.arange(S + 1, dtype=np.int64) * N) // S
    return b[:-1] + (rng.random(S) * (b[1:] - b[:-1])).astype(np.int64)


def simulate_ranks(N: int, S: int, t: int, trials: int, rng: np.random.Generator,
                   placement: str = "random") -> np.ndarray:
    """R for `trials` independent runs (array of int64).

    placement = "random": ranks are a uniformly random permutation (exchangeable input);
    placement = "sorted": rank of position p is N - p (ascending-sorted input, the best
    elements all sit in the last strata).
    """
    out = np.empty(trials, dtype=np.int64)
    for i in range(trials):
        pos = stratified_positions(N, S, rng)
        if placement == "random":
            ranks = rng.permutation(N)[pos] + 1
        elif placement == "sorted":
            ranks = N - pos
        else:
            raise ValueError(placement)
        out[i] = np.partition(ranks, t - 1)[t - 1]
    return out


def failure_rate_exchangeable(N: int, S: int, t: int, k: int, M: int, trials: int,
                              rng: np.random.Generator) -> tuple[float, float]:
    """(Pr(R < k), Pr(R > M)) estimated by drawing the two hypergeometric counts."""
    fail_a = 0.0
    if k > 1:
        x = rng.hypergeometric(k - 1, N - (k - 1), S, size=trials)
        fail_a = float(np.mean(x >= t))
    fail_b = 0.0
    if M < N:
        y = rng.hypergeometric(M, N - M, S, size=trials)
        fail_b = float(np.mean(y <= t - 1))
    return fail_a, fail_b
