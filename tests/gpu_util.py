"""Helpers shared by the GPU parity tests (marshalling between numpy and device tensors only)."""
import numpy as np
import torch

from paper_2609_21594_b200 import workloads as wl

QUINTIC = wl.QUINTIC


def rel(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def dev_f32(x):
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()


def dev_bf16_from_bits(bits):
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


def host_f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def bf16_input(x_f32):
    """fp32 numpy array -> (device bf16 tensor, float64 numpy array of the same bf16 values)."""
    bits = wl.to_bf16_bits(x_f32)
    return dev_bf16_from_bits(bits).reshape(x_f32.shape), wl.bf16_bits_to_f32(bits).astype(np.float64).reshape(x_f32.shape)
