"""Device plumbing around the binding: upload a workload's stored tensors with PyTorch, hand
their pointers to the library, fetch results.  No arithmetic happens here."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B

_TORCH = {"f32": torch.float32, "bf16": torch.bfloat16}


def to_device(t, device="cuda"):
    """workload Tensor (store = float32 or bf16 bit patterns) -> torch tensor on the device."""
    if t.dtype == "bf16":
        return torch.from_numpy(t.store.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(t.store).to(device)        # fp32 as float32, fp8 as its bytes (uint8)


def to_host_f64(x: torch.Tensor) -> np.ndarray:
    """Device tensor -> float64 numpy (exact widening)."""
    return x.detach().to("cpu").to(torch.float64).numpy()


class DeviceWorkload:
    """A workload resident on one GPU and bound to an mk module."""

    def __init__(self, ctx: B.Context, w, weight_layout=B.MK_LAYOUT_TRANSPOSED, device="cuda"):
        self.w = w
        self.ctx = ctx
        self.device = device
        self.dtype = w.dtype
        self.inputs = {k: to_device(t, device) for k, t in w.inputs.items()}
        self.params = {}
        linear_weights = {op["params"]["w"] for op in w.ops if op["kind"] in ("linear", "linear_fp8")}
        for k, t in w.params.items():
            d = to_device(t, device)
            if k in linear_weights and weight_layout == B.MK_LAYOUT_TRANSPOSED:
                d = d.t().contiguous()          # storage layout only: [N, K] row-major
            self.params[k] = (d, t.shape)
        self.module = B.Module(ctx, w.ops, {k: (t.dtype, t.shape) for k, t in w.inputs.items()},
                               weight_layout)
        self.module.set_params(self.params, w.dtype, {k: t.dtype for k, t in w.params.items()})
        out_dt, out_shape, _ = self.module.value_spec(w.ops[-1]["out"])
        self.out = torch.empty(out_shape, dtype=torch.float32 if out_dt == B.MK_F32 else torch.bfloat16, device=device)
        self.ws = None
        self.ws_bytes = 0

    def ensure_workspace(self):
        need = self.module.workspace_size()
        if self.ws is None or need > self.ws_bytes:
            self.ws = torch.empty(max(need, 256), dtype=torch.uint8, device=self.device)
            self.ws_bytes = need
        return need

    def forward(self, stream=None):
        self.ensure_workspace()
        s = torch.cuda.current_stream().cuda_stream if stream is None else stream
        self.module.forward([self.inputs[k] for k in self.module.input_names], self.out, self.ws,
                            self.ws_bytes, s)
        return self.out

    def forward_sub(self, first_sub, count=1, stream=None):
        """Submodules [first_sub, first_sub + count) alone, on what an earlier whole forward left in the workspace."""
        self.ensure_workspace()
        s = torch.cuda.current_stream().cuda_stream if stream is None else stream
        self.module.forward_sub([self.inputs[k] for k in self.module.input_names], self.out, first_sub, count, self.ws,
                                self.ws_bytes, s)
        return self.out

    def swap(self, iters=5, tau=0.9):
        """Rebind submodules that run slower than tau x their fastest alternative (the output tensor is
        overwritten with the result of the final composition)."""
        self.ensure_workspace()
        s = torch.cuda.current_stream().cuda_stream
        r = self.module.swap([self.inputs[k] for k in self.module.input_names], self.out, self.ws, self.ws_bytes, s, iters, tau)
        self.ensure_workspace()
        return r

    def profile(self, iters=10):
        self.ensure_workspace()
        s = torch.cuda.current_stream().cuda_stream
        return self.module.profile([self.inputs[k] for k in self.module.input_names], self.out, self.ws,
                                   self.ws_bytes, s, iters)

    def intermediate(self, name):
        ptr, (dt, shape, _) = self.module.intermediate(name)
        n = int(np.prod(shape))
        esz = 4 if dt == B.MK_F32 else 2
        off = ptr - self.ws.data_ptr()
        assert 0 <= off and off + n * esz <= self.ws.numel()
        raw = self.ws[off: off + n * esz]
        return raw.view(torch.float32 if dt == B.MK_F32 else torch.bfloat16).view(*shape)
