"""Device-side plumbing shared by the tests, the smoke check and the benchmark:
uploads a synthetic problem with torch, creates a context, runs one pass.
No arithmetic of the method happens here."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

from . import binding as B
from .inputs import Dispatched, MoEInputs, MoEShape


def bits_to_device(a: np.ndarray, device) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor on the device."""
    t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
    return t.to(device)


def device_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


@dataclass
class DeviceProblem:
    shape: MoEShape
    M: int
    x: torch.Tensor
    expert_counts: torch.Tensor
    src_rank: torch.Tensor
    src_token: torch.Tensor
    gate: torch.Tensor
    w1: torch.Tensor
    w2: torch.Tensor
    ret: torch.Tensor                 # [R, T*kmax, d]
    out: torch.Tensor                 # [R*T, d]
    slot_out: torch.Tensor
    rows_per_rank_out: torch.Tensor
    segs_per_rank_out: torch.Tensor


def upload(inp: MoEInputs, dsp: Dispatched, device="cuda:0", w1: Optional[torch.Tensor] = None,
           w2: Optional[torch.Tensor] = None) -> DeviceProblem:
    sh = inp.shape
    dev = torch.device(device)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, np.int32)).to(dev)
    M = dsp.M
    return DeviceProblem(
        shape=sh, M=M,
        x=bits_to_device(dsp.x_rows.reshape(M, sh.d), dev) if M else torch.zeros((0, sh.d), dtype=torch.bfloat16, device=dev),
        expert_counts=i32(dsp.expert_counts), src_rank=i32(dsp.src_rank), src_token=i32(dsp.src_token),
        gate=torch.from_numpy(np.ascontiguousarray(dsp.gate, np.float32)).to(dev),
        w1=bits_to_device(inp.w1, dev) if w1 is None else w1,
        w2=(bits_to_device(inp.w2, dev) if inp.w2.size else None) if w2 is None else w2,
        ret=torch.full((sh.R, sh.T * sh.kmax, sh.dout), float("nan"), dtype=torch.bfloat16, device=dev),
        out=torch.full((sh.R * sh.T, sh.dout), float("nan"), dtype=torch.bfloat16, device=dev),
        slot_out=torch.full((max(M, 1),), -7, dtype=torch.int32, device=dev),
        rows_per_rank_out=torch.full((sh.R,), -7, dtype=torch.int32, device=dev),
        segs_per_rank_out=torch.full((sh.R,), -7, dtype=torch.int32, device=dev),
    )


def make_context(shape: MoEShape, max_rows: int, device: int = 0, **kw) -> B.MoeOvl:
    cfg = B.make_config(device=device, num_src_ranks=shape.R, self_rank=shape.self_rank, tokens_per_rank=shape.T,
                        num_local_experts=shape.El, top_k=shape.k, d_model=shape.d, d_ffn=shape.F,
                        single_gemm_out=shape.N_out, max_rows=max_rows, **kw)
    return B.MoeOvl(cfg)


def run(ctx: B.MoeOvl, prob: DeviceProblem, mode: int = B.MODE_OVERLAP, consumer_sm_count: int = 8) -> None:
    ctx.moe_ovl_expert_return(x=prob.x, expert_counts=prob.expert_counts, src_rank=prob.src_rank,
                              src_token=prob.src_token, gate=prob.gate, w1=prob.w1, w2=prob.w2, ret=prob.ret,
                              out=prob.out, consumer_sm_count=consumer_sm_count, mode=mode,
                              slot_out=prob.slot_out, rows_per_rank_out=prob.rows_per_rank_out,
                              segs_per_rank_out=prob.segs_per_rank_out, num_rows=prob.M)
