"""Helpers shared by the GPU parity tests: host numpy <-> device torch conversions."""
import numpy as np
import torch

from paper_2608_04962_b200 import binding as S


def dev_bf16(bits):
    return S.bf16_tensor(bits, "cuda")


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.detach().cpu().numpy()
