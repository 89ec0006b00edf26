"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch


def T(a, device="cuda"):
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def N(t):
    return t.detach().cpu().numpy()
