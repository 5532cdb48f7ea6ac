"""Oracle-side set-up for a named workload -- TEST INFRASTRUCTURE (see cr_oracle.py).

Builds the oracle's own code object and allocation for a workload description
(`n, L, s, P, code, seed`); nothing here comes from the CUDA library.
"""
from __future__ import annotations

from . import cr_oracle as O


def code_for(cfg: dict) -> O.Code:
    n, L, s = cfg["n"], cfg["L"], cfg["s"]
    if cfg["code"] == "printed_3_1":
        return O.Code(n, L, s, [O.printed_code_3_1()[1]] * L, kind="printed")
    if cfg["code"] == "repetition":
        return O.Code(n, L, s, [O.fractional_repetition_code(n, s)] * L, kind="repetition")
    if cfg["code"] == "cyclic":
        B, _ = O.cyclic_random_code(n, s, cfg.get("code_seed", 0), cfg.get("max_kappa", 100.0))
        return O.Code(n, L, s, [B] * L, kind="solve")
    raise ValueError(cfg["code"])


def setup(cfg: dict):
    """(code, local, slot_partition): local[v] = node v's (partition, coefficient) pairs,
    slot_partition = [N][m] nested list of partition ids."""
    code = code_for(cfg)
    local, _ = O.allocate(cfg["n"], cfg["L"], cfg["s"], cfg["P"], code.B_levels)
    return code, local, [[p for p, _ in pairs] for pairs in local]
