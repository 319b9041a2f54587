"""Helpers shared by the GPU parity tests (imported only from tests)."""
import numpy as np
import torch

from paper_2305_12356_b200 import binding as B

ORC_FMT = {}


def orc_fmt(orc, name):
    return getattr(orc, name)


def orc_gran(orc, g):
    return {"tensor": orc.PER_TENSOR, "channel": orc.PER_CHANNEL, "group": orc.PER_GROUP}[g]


def host(x):
    return x.detach().cpu()


def unpack_codes(codes_u8, bits, n):
    c = codes_u8.cpu().numpy()
    if bits == 8:
        return c[:n]
    out = np.empty(2 * c.size, np.uint8)
    out[0::2] = c & 0xF
    out[1::2] = c >> 4
    return out[:n]


def rel_err(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return np.abs(a - b) / np.maximum(np.abs(b), 1e-300)
