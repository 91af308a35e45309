"""Device placement of the seeded inputs: host fp32 arrays -> CUDA tensors in the workload's storage
type.  No arithmetic of the method; used by the tests and by the benchmark."""
from __future__ import annotations

import numpy as np

from . import to_bf16_bits


def to_dev(arr, dtype: str):
    """fp32 host array -> CUDA tensor, bf16 (round to nearest even, the same bits the oracle's inputs hold) or fp32."""
    import torch
    arr = np.ascontiguousarray(arr, dtype=np.float32)
    if dtype == "bf16":
        return torch.from_numpy(to_bf16_bits(arr).view(np.int16).reshape(arr.shape)).view(torch.bfloat16).cuda()
    return torch.from_numpy(arr).cuda()


def dev_weights(W, dtype: str):
    return {n: to_dev(v, dtype) for n, v in W.items() if v is not None}
