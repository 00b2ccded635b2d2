"""Token-sharded (data-parallel) use of the path: the only two places where ranks must talk.

The path splits along tokens: compress, reconstruct, the forward product and the input gradient are
per-token.  Two sums run over tokens and therefore over ranks:

* the sub-token sum behind ``v`` (Section 3.2: the average is over the whole first batch), Dsub floats;
* the weight gradient.  Because ``v`` is shared, ranks can add the factor ``P = dY^T Z`` (O*M floats)
  instead of ``dW`` (O*D values) and expand locally -- Dsub times less traffic.

Both are plain all-reduces (NCCL over NVLink on GPUs, gloo on CPU); nothing here is a kernel.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


def allreduce_sum_(t: torch.Tensor, group=None) -> torch.Tensor:
    """In-place SUM over the ranks of ``group`` (identity without a process group)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t


def sharded_init_v(X_local: torch.Tensor, Dsub: int, ws: Optional[torch.Tensor] = None, group=None) -> torch.Tensor:
    """``v`` of the whole batch from this rank's rows of it: local sum, all-reduce, normalise."""
    from . import binding
    s = binding.velora_subtoken_sum(X_local, Dsub, ws=ws)
    allreduce_sum_(s, group)
    return binding.velora_normalize_v(s)


def sharded_weight_grad(dY_local: torch.Tensor, Z_local: torch.Tensor, v: torch.Tensor, D: int,
                        dW: Optional[torch.Tensor] = None, dw_dtype=torch.bfloat16, beta: int = 0,
                        ws: Optional[torch.Tensor] = None, group=None) -> torch.Tensor:
    """dW of the whole batch: local factor P, all-reduce of P, one local expansion."""
    from . import binding
    P = binding.velora_weight_grad_p(dY_local, Z_local, D, v.shape[0], ws=ws)
    allreduce_sum_(P, group)
    return binding.velora_expand_p(P, v, D, dW=dW, dw_dtype=dw_dtype, beta=beta)
