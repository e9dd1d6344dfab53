"""Device-side convenience around :class:`binding.Plan`: one plan per segment of a workload.

torch is used for device / pinned memory and streams only; every operator runs in the C-ABI
library.  A workload is any object with ``dtype, N, H, W, C, segments`` whose layers carry the
lop_layer fields plus numpy ``weight / scale / shift`` (see the ``lop_inputs`` package).
"""
from types import SimpleNamespace

import numpy as np
import torch

from . import binding as B

_FIELDS = ("op", "cin", "cout", "kh", "kw", "sh", "sw", "ph", "pw", "dh", "dw", "act", "input_from",
           "residual_from", "residual_pos")


def to_device(a, dtype, device):
    """float32 numpy array -> device tensor in the storage dtype (bf16 values must be representable)."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    if dtype == "bf16":
        t = t.to(torch.bfloat16)            # exact: the generators hand out bf16-representable values
    return t.to(device).contiguous()


def to_host_f32(t):
    return t.detach().to("cpu", torch.float32).numpy()


class DeviceChain:
    def __init__(self, wl, flags=0, device="cuda:0", n_bands=None):
        if not torch.cuda.is_available():
            raise RuntimeError("DeviceChain needs a CUDA device; there is no CPU path")
        self.wl, self.device = wl, torch.device(device)
        self.dtype = B.LOP_BF16 if wl.dtype == "bf16" else B.LOP_F32
        self.tdtype = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
        self.keep = []                       # device tensors the plans point into
        self.per_plan = False                # set once the library declines to run the plans as one chain
        self.plans, self.ws, self.outs = [], [], []
        H, W, C = wl.H, wl.W, wl.C
        with torch.cuda.device(self.device):
            for seg in wl.segments:
                layers = []
                for l in seg.layers:
                    d = SimpleNamespace(**{f: getattr(l, f) for f in _FIELDS})
                    d.weight_ptr = d.scale_ptr = d.shift_ptr = None
                    if l.weight is not None:
                        w = to_device(l.weight, wl.dtype, self.device)
                        self.keep.append(w)
                        d.weight_ptr = w.data_ptr()
                    for name in ("scale", "shift"):
                        v = getattr(l, name)
                        if v is not None:
                            t = torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32)).to(self.device)
                            self.keep.append(t)
                            setattr(d, name + "_ptr", t.data_ptr())
                    layers.append(d)
                if n_bands is None:
                    nb = seg.n_bands
                elif isinstance(n_bands, (list, tuple)):                 # one count per segment
                    nb = n_bands[len(self.plans)]
                else:
                    nb = n_bands
                plan = B.Plan(layers, wl.N, H, W, C, self.dtype, nb, flags)
                self.plans.append(plan)
                self.ws.append(torch.zeros(max(plan.workspace_bytes(), 256), dtype=torch.uint8, device=self.device))
                H, W, C = plan.out_shape(plan.num_layers() - 1)
                self.outs.append(torch.zeros((wl.N, H, W, C), dtype=self.tdtype, device=self.device))
        self.staging = torch.zeros((wl.N, wl.H, wl.W, wl.C), dtype=self.tdtype, device=self.device)

    # -- helpers -------------------------------------------------------------------------------
    def input_tensor(self, x=None):
        return to_device(self.wl.x if x is None else x, self.wl.dtype, self.device)

    def pinned_input(self, x=None):
        t = torch.from_numpy(np.ascontiguousarray(self.wl.x if x is None else x, dtype=np.float32))
        if self.wl.dtype == "bf16":
            t = t.to(torch.bfloat16)
        return t.contiguous().pin_memory()

    def _stream(self, stream):
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        return s.cuda_stream

    def layer_output(self, seg, layer):
        """The full-size output tensor of one layer of a segment: the segment's output tensor for its last layer, else a
        view into the segment's workspace (lop_plan_layer_offset).  None when executions never write it (a convolution
        whose pooling is folded into its epilogue, lop_plan_layer_stored)."""
        plan = self.plans[seg]
        if layer == plan.num_layers() - 1:
            return self.outs[seg]
        if not plan.layer_stored(layer):
            return None
        h, w, c = plan.out_shape(layer)
        n = self.wl.N * h * w * c
        off = plan.layer_offset(layer)
        es = 2 if self.wl.dtype == "bf16" else 4
        return self.ws[seg][off:off + n * es].view(self.tdtype).view(self.wl.N, h, w, c)

    # -- execution -----------------------------------------------------------------------------
    def run_whole(self, x_dev, stream=None):
        s = self._stream(stream)
        for plan, ws, out in zip(self.plans, self.ws, self.outs):
            plan.run_whole(x_dev.data_ptr(), out.data_ptr(), ws.data_ptr(), s)
            x_dev = out
        return self.outs[-1]

    def _chain(self):
        """Several tensor-core plans run as one launch; False when the library wants them one by one."""
        return len(self.plans) > 1 and not self.per_plan

    def run_banded(self, x_dev, stream=None):
        s = self._stream(stream)
        if self._chain():
            try:
                B.run_chain_banded(self.plans, x_dev.data_ptr(), [o.data_ptr() for o in self.outs], [w.data_ptr() for w in self.ws], s)
                return self.outs[-1]
            except B.LopError as e:
                if e.status != -3:
                    raise
                self.per_plan = True
        for plan, ws, out in zip(self.plans, self.ws, self.outs):
            plan.run_banded(x_dev.data_ptr(), out.data_ptr(), ws.data_ptr(), s)
            x_dev = out
        return self.outs[-1]

    def run_bands_one_by_one(self, x_dev, order=None, stream=None):
        s = self._stream(stream)
        for plan, ws, out in zip(self.plans, self.ws, self.outs):
            for b in (range(plan.num_bands()) if order is None else order(plan.num_bands())):
                plan.run_band(b, x_dev.data_ptr(), out.data_ptr(), ws.data_ptr(), s)
            x_dev = out
        return self.outs[-1]

    def run_pipelined(self, x_pinned, stream=None, out_pinned=None):
        """Segment 0 streams its input bands from pinned host memory; later segments run band-wise on the device.

        out_pinned: a pinned host tensor of the last output's shape; the last layer's kernels then store the result
        straight into it (every execution call takes device-addressable host memory as its output tensor)."""
        s = self._stream(stream)
        outs = [o.data_ptr() for o in self.outs]
        if out_pinned is not None:
            outs[-1] = out_pinned.data_ptr()
        if self._chain():
            try:
                B.run_chain_pipelined(self.plans, x_pinned.data_ptr(), self.staging.data_ptr(), outs, [w.data_ptr() for w in self.ws], s)
                return self.outs[-1] if out_pinned is None else out_pinned
            except B.LopError as e:
                if e.status != -3:
                    raise
                self.per_plan = True
        self.plans[0].run_pipelined(x_pinned.data_ptr(), self.staging.data_ptr(), outs[0], self.ws[0].data_ptr(), s)
        for i in range(1, len(self.plans)):
            self.plans[i].run_banded(outs[i - 1], outs[i], self.ws[i].data_ptr(), s)
        return self.outs[-1] if out_pinned is None else out_pinned

    def check_device(self):
        for plan, ws in zip(self.plans, self.ws):
            plan.check_device(ws.data_ptr())

    def launches(self):
        return sum(p.last_launches() for p in self.plans)

    def flops(self):
        return sum(p.flops() for p in self.plans)
