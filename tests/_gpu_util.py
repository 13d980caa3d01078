"""Helpers shared by the GPU parity tests: move numpy arrays to the device and back."""
import numpy as np
import torch


def dev_f32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def dev_bf16(bits):
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor on the device."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def dev_u32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint32).view(np.int32)).cuda()


def host_u32(t):
    return t.cpu().numpy().view(np.uint32)


def host_bf16_bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def workspace(nbytes):
    return torch.empty((nbytes + 255) // 256 * 256, dtype=torch.uint8, device="cuda")
