"""One UoE transformer block with preallocated buffers: the forward is the single C entry point
uoe_block_forward, the backward the per-half entry points.

u = SMHA(h) (router, Eq. 27-36), out = UoME(u) (router, Eq. 37-40): each sub-block has its own router,
as in Section III-C.  Nothing is computed here; the class only owns device buffers and issues the calls.
"""
from __future__ import annotations

import torch

from . import binding as B


class UoEBlock:
    def __init__(self, prob_att: B.Problem | None, prob_mlp: B.Problem | None, weights: dict, device="cuda",
                 save_h: bool = False, backward: bool = False):
        self.pa, self.pm, self.w = prob_att, prob_mlp, weights
        p0 = prob_att or prob_mlp
        self.u = torch.empty(p0.B, p0.L, p0.d, dtype=p0.torch_dtype, device=device)
        self.out = torch.empty_like(self.u)
        self.ws_blk = B.alloc_block_workspace(prob_att, prob_mlp, device)
        if prob_att is not None:
            self.ra = B.alloc_routing(prob_att, device)
            self.ws_ra = B.alloc_workspace(prob_att, B.UOE_OP_ROUTE, device)
            if backward:          # SMHA backward buffers (Eq. 27-36 differentiated)
                f32 = torch.float32
                self.ws_ab = B.alloc_workspace(prob_att, B.UOE_OP_SMHA_BWD, device)
                self.dh = torch.empty_like(self.u)
                self.dWa = {k: torch.empty(weights[k].shape, dtype=f32, device=device)
                            for k in ("Wq", "Wk", "Wv", "Wo", "Wr_att")}
        if prob_mlp is not None:
            self.rm = B.alloc_routing(prob_mlp, device)
            self.ws_rm = B.alloc_workspace(prob_mlp, B.UOE_OP_ROUTE, device)
            self.saved_h = B.alloc_saved_h(prob_mlp, device) if (save_h or backward) else None
            self.backward = backward
            if backward:          # UoME backward buffers (Eq. 38-40 differentiated)
                f32 = torch.float32
                self.ws_b = B.alloc_workspace(prob_mlp, B.UOE_OP_MLP_BWD, device)
                self.dx = torch.empty_like(self.u)
                self.dW1 = torch.empty(weights["W1"].shape, dtype=f32, device=device)
                self.dW2 = torch.empty(weights["W2"].shape, dtype=f32, device=device)
                self.dWr = torch.empty(weights["Wr_mlp"].shape, dtype=f32, device=device)

    def forward(self, h: torch.Tensor, check: bool = False) -> torch.Tensor:
        """The whole block through uoe_block_forward; the routing of both halves is kept for the backward."""
        both = self.pa is not None and self.pm is not None
        return B.uoe_block_forward(self.pa, self.pm, h, self.w, r_att=getattr(self, "ra", None),
                                   r_mlp=getattr(self, "rm", None), u=self.u if both else None, y=self.out,
                                   saved_h=getattr(self, "saved_h", None), ws=self.ws_blk, check=check)

    def mlp_backward(self, h: torch.Tensor, dy: torch.Tensor, check: bool = False):
        """Backward of the UoME half for the routing and saved pre-activations of the last forward(h)."""
        w = self.w
        return B.uoe_mlp_backward(self.pm, h, w["W1"], w["W2"], w["Wr_mlp"], self.rm, self.saved_h, dy, dx=self.dx,
                                  dW1=self.dW1, dW2=self.dW2, dW_r=self.dWr, ws=self.ws_b, check=check)

    def smha_backward(self, h: torch.Tensor, du: torch.Tensor, check: bool = False):
        """Backward of the SMHA half for the routing of the last forward(h); du is the gradient w.r.t. its output."""
        w, g = self.w, self.dWa
        return B.uoe_smha_backward(self.pa, h, w["Wq"], w["Wk"], w["Wv"], w["Wo"], w["Wr_att"], self.ra, du, dx=self.dh,
                                   dWq=g["Wq"], dWk=g["Wk"], dWv=g["Wv"], dWo=g["Wo"], dW_r=g["Wr_att"], ws=self.ws_ab,
                                   check=check)

    def device_status(self) -> int:
        worst = 0
        for name in ("ws_blk", "ws_ra", "ws_rm", "ws_b", "ws_ab"):
            ws = getattr(self, name, None)
            if ws is not None:
                worst = max(worst, B.uoe_read_device_status(ws))
        return worst
