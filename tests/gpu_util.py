"""Helpers for the GPU parity tests: move a host problem onto the device, run the
library through its C ABI (via the thin binding) and hand back numpy results."""
from __future__ import annotations

import os

import numpy as np
import torch

import paper_2608_05483_b200 as P

DEV = "cuda:0"


def bits_to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 patterns -> bf16 device tensor with the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(DEV).view(torch.bfloat16)


class Runner:
    """One context + one registered pool built from host-side logical matrices."""

    def __init__(self, prob, max_tokens=None, layer=0, proj=0, on_device=False):
        self.prob = prob
        self.layer, self.proj = layer, proj
        self.ctx = P.Context(max_tokens or max(1, prob["T"]), prob["N"])
        if prob.get("fp16"):
            self.ctx.set_input_type(True)     # the 16-bit patterns are IEEE half; device tensors keep a bf16 label
        if os.environ.get("PLORA_TEST_INPUTS_RESIDENT") == "1":
            # the tests' x is on the device long before any call: every case may also run under the hint
            self.ctx.set_inputs_resident(True)
        if on_device:
            A = [bits_to_dev(a) for a in prob["A"]]
            B = [bits_to_dev(b) for b in prob["B"]]
        else:
            A, B = prob["A"], prob["B"]
        self.slab = self.ctx.register_pool(layer, proj, prob["d_in"], prob["d_out"], prob["ranks"], prob["scales"], A, B)
        self.x = bits_to_dev(prob["x"]) if prob["T"] else torch.empty((0, prob["d_in"]), dtype=torch.bfloat16, device=DEV)
        self.ids = torch.from_numpy(prob["ids"]).to(DEV)

    def delta(self, path=P.PATH_FUSED, y_in=None, ids=None, guard=True):
        p = self.prob
        T, d_out = p["T"], p["d_out"]
        self.ctx.set_path(path)
        # one guard row on each side of y catches writes outside the output
        buf = torch.full((T + 2, d_out), 12345.0, dtype=torch.float32, device=DEV)
        y = buf[1:T + 1]
        if y_in is None:
            y.zero_()
        else:
            y.copy_(torch.from_numpy(y_in))
        ids_t = self.ids if ids is None else torch.from_numpy(np.ascontiguousarray(ids, np.int32)).to(DEV)
        self.ctx.bucket(ids_t, p["N"])
        self.ctx.lora_delta(self.x, ids_t, self.layer, self.proj, y)
        torch.cuda.synchronize()
        out = buf.cpu().numpy()
        if guard:
            assert np.all(out[0] == 12345.0) and np.all(out[-1] == 12345.0), "guard rows of y were written"
        return out[1:T + 1].copy()

    def close(self):
        self.ctx.close()
