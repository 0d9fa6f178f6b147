"""Host-fed forward passes with the copies overlapped.

A caller whose activations live in host memory pays, per step, a host-to-device copy of x, the
forward pass, and a device-to-host copy of the result.  Run back to back on one stream the three
add up (at the 262M-scale shape: ~0.3 ms + 0.12 ms + ~0.6 ms over PCIe); HostFedLayer runs them on
three streams with two device buffers each for x and out, so that step i's result goes back to the
host while step i + 1 computes and step i + 2's input arrives: the steady-state time per step is
that of the slowest of the three.  Argument marshalling and stream plumbing only: every step of
the layer itself runs in the library's kernels (binding.Layer.sh_forward).
"""
from __future__ import annotations

import torch

from . import binding


class HostFedLayer:
    def __init__(self, layer: "binding.Layer", like_x: torch.Tensor):
        """layer: a configured binding.Layer with its weights set; like_x: a device tensor with the
        shape and dtype of the layer's input."""
        self.layer = layer
        dev = like_x.device
        self.x_dev = [torch.empty_like(like_x) for _ in range(2)]
        # (the layer's output dtype: fp32, or fp16 after sh_set_output_f16 - half the bytes on the way back)
        self.out_dev = [torch.empty(like_x.shape, dtype=getattr(layer, "out_dtype", torch.float32), device=dev) for _ in range(2)]
        self.s_in, self.s_compute, self.s_out = (torch.cuda.Stream(device=dev) for _ in range(3))
        mk = lambda: [torch.cuda.Event() for _ in range(2)]
        self.ev_in, self.ev_computed, self.ev_out = mk(), mk(), mk()
        self.step_no = 0
        for st in (self.s_in, self.s_compute, self.s_out):      # after whatever set the layer up
            st.wait_stream(torch.cuda.current_stream(dev))

    def step(self, x_host: torch.Tensor, out_host: torch.Tensor) -> None:
        """Enqueue one step: x_host (pinned) -> device, forward, result -> out_host (pinned).
        Returns at once; out_host is valid after wait() (or once a later step has reused its slot).
        The caller alternates between two out_host buffers or consumes one before the step after next."""
        s = self.step_no & 1
        first_use = self.step_no < 2
        with torch.cuda.stream(self.s_in):
            if not first_use:
                self.s_in.wait_event(self.ev_computed[s])       # the pass that read x_dev[s] is done
            self.x_dev[s].copy_(x_host, non_blocking=True)
            self.ev_in[s].record(self.s_in)
        with torch.cuda.stream(self.s_compute):
            self.s_compute.wait_event(self.ev_in[s])
            if not first_use:
                self.s_compute.wait_event(self.ev_out[s])       # out_dev[s] has been copied out
            self.layer.sh_forward(self.x_dev[s], self.out_dev[s])
            self.ev_computed[s].record(self.s_compute)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_computed[s])
            out_host.copy_(self.out_dev[s], non_blocking=True)
            self.ev_out[s].record(self.s_out)
        self.step_no += 1

    def wait(self) -> None:
        for st in (self.s_in, self.s_compute, self.s_out):
            st.synchronize()
