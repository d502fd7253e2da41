"""Helpers for the GPU parity tests: run a synthetic workload through the C ABI with torch tensors
as device buffers (torch is only the allocator here)."""
import numpy as np
import torch

import paper_2207_05022_b200 as sti
from oracle import sti_oracle as O

REL_TOL = 2e-2          # max|y - y_ref| / max|y_ref|, bf16 operands with fp32 accumulation


def to_device_act(work, x_dev_np=None):
    a = work.x_dev if x_dev_np is None else x_dev_np
    if work.act_dtype == "bf16":
        return torch.from_numpy(a.view(np.int16).copy()).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def from_device_act(t):
    return t.float().cpu().numpy().astype(np.float64)


def rel_err(y, ref):
    return float(np.abs(y - ref).max() / np.abs(ref).max())


def run_model(sess, work, host=False, lens=None):
    x = to_device_act(work)
    y = torch.empty_like(x)
    lens_dev = 0
    keep = None
    if lens is not None:
        keep = torch.tensor(lens, dtype=torch.int32).cuda()
        lens_dev = keep.data_ptr()
    torch.cuda.synchronize()
    if host:
        xh = x.cpu().pin_memory()
        yh = torch.empty_like(xh).pin_memory()
        lens_h = None if lens is None else np.asarray(lens, dtype=np.int32)
        sti.sti_model_forward_host(sess.plan, xh.data_ptr(), yh.data_ptr(), work.batch, work.seq,
                                   0 if lens_h is None else lens_h.ctypes.data)
        sti.sti_sync(sess.ctx)
        return from_device_act(yh)
    sti.sti_model_forward(sess.plan, x.data_ptr(), y.data_ptr(), work.batch, work.seq, lens_dev)
    sti.sti_sync(sess.ctx)
    return from_device_act(y)


def run_layer(sess, work, layer, x_np_values=None, lens=None):
    x = to_device_act(work) if x_np_values is None else x_np_values
    y = torch.empty_like(x)
    lens_dev = 0
    keep = None
    if lens is not None:
        keep = torch.tensor(lens, dtype=torch.int32).cuda()
        lens_dev = keep.data_ptr()
    torch.cuda.synchronize()
    sti.sti_layer_forward(sess.plan, layer, x.data_ptr(), y.data_ptr(), work.batch, work.seq, lens_dev)
    sti.sti_sync(sess.ctx)
    return from_device_act(y)
