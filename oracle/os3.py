"""CPU oracle for the optimal speculation stride scheduler (OS^3). Test infrastructure only:
nothing in the product path may import it; it shares no code with the library.

Written from Section 4 ("Optimal speculation stride scheduler") and Appendix A.2 of the paper
in plain Python floats (fp64), one function per formula, no closed-form shortcuts:

  expected_verified   the sum of gamma^i over i = 0..s-1 (the last-but-one line of the
                      appendix derivation), term by term
  objective           expected verified documents per unit time, synchronous or asynchronous
  estimate_gamma      the windowed maximum-likelihood estimate, truncated at gamma_max
  best_stride         exhaustive argmax over 1..s_max (first maximum wins)
"""


def expected_verified(gamma: float, s: int) -> float:
    total = 0.0
    for i in range(s):
        total += gamma ** i
    return total


def latency(gamma: float, a: float, b: float, s: int, async_verify: bool) -> float:
    sync = s * a + b
    if not async_verify:
        return sync
    p_all = gamma ** s
    return p_all * ((s - 1) * a + max(a, b)) + (1.0 - p_all) * sync


def objective(gamma: float, a: float, b: float, s: int, async_verify: bool) -> float:
    return expected_verified(gamma, s) / latency(gamma, a, b, s, async_verify)


def estimate_gamma(matched, strides, gamma_max: float) -> float:
    hits = sum(int(m) for m in matched)
    misses = sum(1 for m, s in zip(matched, strides) if int(m) < int(s))
    if hits + misses == 0:
        return 0.0
    return min(hits / (hits + misses), gamma_max)


def best_stride(matched, strides, gamma_max: float, a: float, b: float, s_max: int,
                async_verify: bool) -> int:
    g = estimate_gamma(matched, strides, gamma_max)
    best_s, best_v = 1, objective(g, a, b, 1, async_verify)
    for s in range(2, s_max + 1):
        v = objective(g, a, b, s, async_verify)
        if v > best_v:
            best_s, best_v = s, v
    return best_s
