"""Reporting formulas (host side, no device work)."""


def step_speedup_bound(r_gen: float, gen_speedup: float) -> float:
    """Upper bound on the speed-up of a whole RL step when only rollout generation gets faster
    (Section 2.2, the Amdahl bound): 1 / (R_gen / s + 1 - R_gen), with R_gen the generation share of the
    step and s the generation speed-up (the mean acceptance length, under the bound's assumption that a
    speculation step costs one autoregressive forward)."""
    return 1.0 / (r_gen / gen_speedup + (1.0 - r_gen))


def expected_tokens_per_step(a: float, k: int) -> float:
    """Mean tokens produced per speculation step under independent per-token acceptance a: (1-a^(k+1))/(1-a)."""
    return float(k + 1) if a >= 1.0 else (1.0 - a ** (k + 1)) / (1.0 - a)
