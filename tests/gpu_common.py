"""Helpers shared by the GPU parity tests (not a test module)."""
import numpy as np
import torch

from oracle import oracle as O
from paper_2609_26077_b200 import fmm, realizations as P

MODES = {"fp32": O.SCALE_FP32, "ue8m0": O.SCALE_UE8M0}


def coeffs(name):
    return (None, None, None) if name == "cubic" else P.get(name)


def make_plan(name, levels, blk, mode):
    U, V, W = coeffs(name)
    return fmm.Plan(U, V, W, levels=0 if name == "cubic" else levels, block_k=blk, scale_mode=mode)


def dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def oracle_scales(scales, e8, mode):
    return scales if mode == "fp32" else e8
