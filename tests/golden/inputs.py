"""Inputs of the stored example: closed-form, no random numbers, none of the method's arithmetic.

q, k, v are sums of two sinusoids in (head, position, channel), rounded to bf16; sized so that the paired
tensor-core kernel runs them (head_dim 128, block 128) and the float64 oracle needs a second."""
import math

import torch

HQ, HKV, N, D, B = 4, 2, 1024, 128, 128
CLUSTER_MAP = [0, 0, 1, 1]
PIVOT_HEADS = [0, 2]
GAMMA = 0.9


def make():
    n = torch.arange(N, dtype=torch.float64).view(1, N, 1)
    c = torch.arange(D, dtype=torch.float64).view(1, 1, D)

    def field(heads, a, b, amp):
        h = torch.arange(heads, dtype=torch.float64).view(heads, 1, 1)
        x = torch.sin(a * (h + 1) + 0.013 * n * (1 + c % 7) + 0.31 * c) + 0.5 * torch.cos(b * n / (1 + c % 5) + 0.7 * h)
        return (amp * x).to(torch.bfloat16)

    q = field(HQ, 0.37, 0.021, 1.6 / math.sqrt(math.sqrt(D)) * 2)
    k = field(HKV, 0.53, 0.017, 1.6 / math.sqrt(math.sqrt(D)) * 2)
    v = field(HKV, 0.71, 0.029, 1.0)
    return q, k, v
