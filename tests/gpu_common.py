"""Helpers shared by the GPU parity tests."""
import numpy as np

from oracle import cr_oracle as O
from oracle import cr_setup
from paper_1902_01981_b200 import binding as B
from paper_1902_01981_b200 import inputs

CODE_ID = {"printed_3_1": B.CR_CODE_PAPER_3_1, "cyclic": B.CR_CODE_CYCLIC_RANDOM,
           "repetition": B.CR_CODE_FRACTIONAL_REPETITION}

# fp32 parity bar: relative L2 error of the CUDA result against the fp64 oracle
REL_L2_BAR = 1e-5


def rel_l2(got, want) -> float:
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    denom = np.linalg.norm(want)
    return float(np.linalg.norm(got - want) / (denom if denom > 0 else 1.0))


def make_plan(cfg, dtype=B.CR_F32, device=0, d=None):
    return B.cr_plan_create(cfg["n"], cfg["L"], cfg["s"], cfg["P"], cfg["d"] if d is None else d,
                            code=CODE_ID[cfg["code"]], dtype=dtype, seed=cfg.get("code_seed", 0),
                            max_kappa=cfg.get("max_kappa", 0.0), device=device)


def slots_on_device(plan, G_parts, torch):
    """Replicates the partition gradients into the [N, m, d] slot buffer on the GPU.  The slot ->
    partition table is checked against the oracle's allocation before it is used."""
    part = B.slot_partitions(plan)
    dev = torch.from_numpy(G_parts).cuda()
    idx = torch.from_numpy(part.astype(np.int64).reshape(-1)).cuda()
    out = dev.index_select(0, idx).reshape(part.shape[0], part.shape[1], G_parts.shape[1]).contiguous()
    return out


def check_slot_table(plan, cfg):
    code, local, slot_part = cr_setup.setup(cfg)
    assert B.slot_partitions(plan).tolist() == slot_part
    return code, local
