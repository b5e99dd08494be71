"""Helpers shared by the GPU parity tests (marshalling between numpy bit patterns and torch)."""
import numpy as np
import torch

import synth


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def dev_i32(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def weights(c, which):
    """bf16 bit patterns of a config's weight matrix (fp32 configs are rounded once, as the library does)."""
    w = synth.gaussian_weights(c["V"], c["d"], c["wstd"], c["wseed"], which, c["wdtype"])
    return synth.f32_to_bf16_bits(w) if c["wdtype"] == "f32" else w
