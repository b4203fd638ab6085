"""torch.optim front ends of the fused 8-bit steps: `SGD8bit` and `AdamW8bit`.

The optimizers of Section IV of the paper ("SGD (8-bit)", "Adam (8-bit)") as drop-in
`torch.optim.Optimizer` classes: the states live as uint8 codes plus one fp32 maximum per block of
`block_size` elements, and `step()` is one launch of the CUDA library per parameter group (the
pointer-list entry points), whatever the number of tensors.  These classes only keep the state
tensors and marshal pointers; all arithmetic runs in `libdt8.so`.

Parameters must be contiguous fp32 or bf16 CUDA tensors (bf16 parameters are stepped without a
32-bit copy: widened, updated in fp32, rounded once on store); gradients fp32 or bf16; one dtype
of each per group.
The pointer arrays are rebuilt only when a parameter's or gradient's address changes, so
`optimizer.zero_grad(set_to_none=False)` keeps the per-step host cost at one launch.
`state_dict()` / `load_state_dict()` carry the codes, the block maxima and the step count, so a
resumed run continues bit-identically.
"""
from __future__ import annotations

from typing import Dict, List

import torch

import paper_2412_01195_b200 as dt8


class _Optimizer8bit(torch.optim.Optimizer):
    _adam = False

    def __init__(self, params, defaults, block_size: int):
        if block_size not in dt8.BLOCK_SIZES:
            raise ValueError(f"block_size must be one of {dt8.BLOCK_SIZES}")
        defaults = dict(defaults, block_size=block_size)
        super().__init__(params, defaults)
        self._prepared: Dict[int, tuple] = {}

    def _state_of(self, p: torch.Tensor, block_size: int) -> dict:
        st = self.state[p]
        if "m_codes" not in st:
            st["m_codes"], st["m_absmax"] = dt8.new_state(p.numel(), block_size, True, p.device)
            if self._adam:
                st["r_codes"], st["r_absmax"] = dt8.new_state(p.numel(), block_size, False, p.device)
        return st

    def _prepare(self, gi: int, group: dict):
        ps: List[torch.Tensor] = [p for p in group["params"] if p.grad is not None]
        if not ps:
            return None
        for p in ps:
            if p.grad.is_sparse:
                raise RuntimeError("sparse gradients are not supported")
            if not (p.is_cuda and p.dtype in (torch.float32, torch.bfloat16) and p.is_contiguous()):
                raise TypeError("parameters must be contiguous float32 or bfloat16 CUDA tensors")
        if any(p.dtype != ps[0].dtype for p in ps):
            raise TypeError("the parameters of one group share a dtype (use one group per dtype)")
        gs = [p.grad if p.grad.is_contiguous() else p.grad.contiguous() for p in ps]
        B = group["block_size"]
        sts = [self._state_of(p, B) for p in ps]
        key = tuple(t.data_ptr() for t in ps) + tuple(g.data_ptr() for g in gs) + \
            tuple(s["m_codes"].data_ptr() for s in sts)
        cached = self._prepared.get(gi)
        if cached is None or cached[0] != key:
            lists = dt8.PreparedTensorList(
                [p.data for p in ps], gs, [s["m_codes"] for s in sts], [s["m_absmax"] for s in sts],
                [s["r_codes"] for s in sts] if self._adam else None,
                [s["r_absmax"] for s in sts] if self._adam else None)
            cached = (key, lists)
            self._prepared[gi] = cached
        return cached[1]

    def load_state_dict(self, state_dict) -> None:
        """torch casts every loaded floating-point state tensor to the parameter's dtype and
        leaves the others alone only by their dtype; the uint8 codes must stay uint8 and the
        block maxima fp32 (also under bf16 parameters), so both are set aside and put back
        untouched."""
        keep = ("_codes", "_absmax")
        held = {}
        stripped = {"param_groups": state_dict["param_groups"], "state": {}}
        for pid, st in state_dict["state"].items():
            stripped["state"][pid] = {k: v for k, v in st.items() if not k.endswith(keep)}
            held[pid] = {k: v for k, v in st.items() if k.endswith(keep)}
        super().load_state_dict(stripped)
        ids = [pid for g in state_dict["param_groups"] for pid in g["params"]]
        params = [p for g in self.param_groups for p in g["params"]]
        for pid, p in zip(ids, params):
            for k, v in held.get(pid, {}).items():
                dtype = torch.uint8 if k.endswith("_codes") else torch.float32
                self.state[p][k] = v.detach().to(device=p.device, dtype=dtype).clone()
        # a state saved with another block size (or for another tensor) must not reach a kernel
        for group in self.param_groups:
            for p in group["params"]:
                st = self.state.get(p, {})
                if "m_codes" not in st:
                    continue
                by_el = {k: st[k] for k in ("m_codes", "r_codes") if k in st}
                by_bl = {k: st[k] for k in ("m_absmax", "r_absmax") if k in st}
                dt8._check_layout("load_state_dict", p.numel(), group["block_size"], p.device, by_el, by_bl)
        self._prepared.clear()

    def state_bytes(self) -> int:
        """Bytes of optimizer state currently held (codes and block maxima)."""
        total = 0
        for st in self.state.values():
            for k in ("m_codes", "m_absmax", "r_codes", "r_absmax"):
                if k in st:
                    total += st[k].numel() * st[k].element_size()
        return total


class SGD8bit(_Optimizer8bit):
    """SGD with momentum whose momentum buffer is stored in 8 bits (Eq. sgd inside Eq. quant1-3).
    Weight decay is the coupled form (added to the gradient), as in torch.optim.SGD."""

    def __init__(self, params, lr: float, momentum: float = 0.9, weight_decay: float = 0.0,
                 block_size: int = 2048):
        super().__init__(params, dict(lr=lr, momentum=momentum, weight_decay=weight_decay, step=0),
                         block_size)

    @torch.no_grad()
    def step(self, closure=None):
        loss = None
        if closure is not None:
            with torch.enable_grad():
                loss = closure()
        for gi, group in enumerate(self.param_groups):
            lists = self._prepare(gi, group)
            if lists is None:
                continue
            group["step"] += 1
            lists.sgd_step(group["lr"], group["momentum"], group["weight_decay"], group["step"],
                           group["block_size"])
        return loss


class AdamW8bit(_Optimizer8bit):
    """Adam / AdamW whose two moments are stored in 8 bits (Eq. adam inside Eq. quant1-3).
    decoupled=True is AdamW (the optimizer the paper trains its DF-ResNets with); decoupled=False
    adds the decay to the gradient (torch.optim.Adam); bias_correction=False gives the equation
    exactly as the paper prints it."""
    _adam = True

    def __init__(self, params, lr: float = 1e-3, betas=(0.9, 0.999), eps: float = 1e-8,
                 weight_decay: float = 0.01, decoupled: bool = True, bias_correction: bool = True,
                 block_size: int = 2048):
        flags = (dt8.DT8_ADAM_DECOUPLED_WD if decoupled else 0) | \
                (dt8.DT8_ADAM_BIAS_CORRECTION if bias_correction else 0)
        super().__init__(params, dict(lr=lr, betas=tuple(betas), eps=eps, weight_decay=weight_decay,
                                      flags=flags, step=0), block_size)

    @torch.no_grad()
    def step(self, closure=None):
        loss = None
        if closure is not None:
            with torch.enable_grad():
                loss = closure()
        for gi, group in enumerate(self.param_groups):
            lists = self._prepare(gi, group)
            if lists is None:
                continue
            group["step"] += 1
            b1, b2 = group["betas"]
            lists.adam_step(group["lr"], b1, b2, group["eps"], group["weight_decay"], group["step"],
                            group["block_size"], group["flags"])
        return loss
