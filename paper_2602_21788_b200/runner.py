"""Device-buffer plumbing around the C ABI for tests, the smoke check and the benchmark: allocates
torch tensors, calls the library, returns numpy results.  No arithmetic of the method happens here."""
from __future__ import annotations

import numpy as np
import torch

from . import fcp, synth


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def bf16_dev_to_f64(t: torch.Tensor) -> np.ndarray:
    """bf16 device tensor -> host array.  float32 holds every bf16 value exactly and halves the host
    memory of the large workloads; numpy promotes to float64 when it is compared with the oracle."""
    return t.float().cpu().numpy()


class DeviceState:
    """All device buffers of one workload (inputs, partials, outputs, scratch) and its uploaded plan."""

    def __init__(self, w: synth.Workload, q, k, v, do=None, heads_per_pass=None, want_o_f32=False, partials=True,
                 kv_heads_per_bwd_pass=None):
        """q, k, v, do: bf16 bit patterns on the host (numpy uint16) or bf16 tensors already on the device.
        `partials=False` skips the partial buffers (enough for the fused forward)."""
        self.w = w
        self.plan = fcp.Plan(w.seqlens, w.cp_degrees, w.hq, w.hkv, w.head_dim, spans=w.spans).upload()
        T, hq, hkv, D = w.total_tokens, w.hq, w.hkv, w.head_dim
        self.hpp = heads_per_pass or hq
        dev = lambda a: a if isinstance(a, torch.Tensor) else to_dev_bf16(a)
        self.q, self.k, self.v = dev(q), dev(k), dev(v)
        self.do = dev(do) if do is not None else None
        R = self.plan.info("R")
        self.R = R
        if partials:
            self.o_part = torch.empty((R, self.hpp, D), dtype=torch.float32, device="cuda")
            self.lse_part = torch.empty((R, self.hpp), dtype=torch.float32, device="cuda")
        self.o = torch.empty((T, hq, D), dtype=torch.bfloat16, device="cuda")
        self.lse = torch.empty((T, hq), dtype=torch.float32, device="cuda")
        self.o_f32 = torch.empty((T, hq, D), dtype=torch.float32, device="cuda") if want_o_f32 else None
        if do is not None:
            self.dq = torch.empty((T, hq, D), dtype=torch.bfloat16, device="cuda")
            self.dk = torch.empty((T, hkv, D), dtype=torch.bfloat16, device="cuda")
            self.dv = torch.empty((T, hkv, D), dtype=torch.bfloat16, device="cuda")
            self.kv_pass = kv_heads_per_bwd_pass or hkv
            self.scratch_bytes = self.plan.bwd_scratch_bytes(self.kv_pass)
            self.scratch = torch.empty(self.scratch_bytes, dtype=torch.uint8, device="cuda")

    def forward(self, stream=None, merged=False):
        """Forward over the plan + merge, in head passes.  `merged` uses the single call that writes
        single-slot chunks straight to the output (no fp32 copy of the output, partials incomplete)."""
        st = (stream or torch.cuda.current_stream()).cuda_stream
        for h0 in range(0, self.w.hq, self.hpp):
            hc = min(self.hpp, self.w.hq - h0)
            if merged:
                fcp.fcp_attn_fwd_merged(self.plan, self.q, self.k, self.v, self.o_part, self.lse_part, self.o, self.lse,
                                        h0, hc, st)
            else:
                fcp.fcp_attn_fwd(self.plan, self.q, self.k, self.v, self.o_part, self.lse_part, h0, hc, st)
                fcp.fcp_lse_merge(self.plan, self.o_part, self.lse_part, self.o, self.lse, h0, hc, st, o_f32=self.o_f32)

    def forward_fused(self, stream=None):
        """Forward with the merge on the fly (no partial buffers), in head passes of `heads_per_pass`."""
        st = (stream or torch.cuda.current_stream()).cuda_stream
        for h0 in range(0, self.w.hq, self.hpp):
            hc = min(self.hpp, self.w.hq - h0)
            fcp.fcp_attn_fwd_fused(self.plan, self.q, self.k, self.v, self.o, self.lse, h0, hc, st, o_f32=self.o_f32)

    def backward(self, stream=None):
        st = (stream or torch.cuda.current_stream()).cuda_stream
        if self.kv_pass == self.w.hkv:
            fcp.fcp_attn_bwd(self.plan, self.q, self.k, self.v, self.o, self.do, self.lse, self.dq, self.dk, self.dv,
                             self.scratch, self.scratch_bytes, st)
            return
        for k0 in range(0, self.w.hkv, self.kv_pass):
            kc = min(self.kv_pass, self.w.hkv - k0)
            fcp.fcp_attn_bwd_heads(self.plan, self.q, self.k, self.v, self.o, self.do, self.lse, k0, kc, self.dq, self.dk,
                                   self.dv, self.scratch, self.scratch_bytes, st)

    def check_status(self):
        st = self.plan.device_status()
        if st[0] != 0:
            raise RuntimeError(f"device status {fcp.status_string(int(st[0]))}: where={st[1]} block={st[2]} thread={st[3]}")


def run_fwd_bwd(w, q, k, v, do=None, heads_per_pass=None, keep_partials=False, want_o_f32=True, fused=False,
                kv_heads_per_bwd_pass=None):
    """`fused`: forward through fcp_attn_fwd_fused instead of fcp_attn_fwd + fcp_lse_merge."""
    ds = DeviceState(w, q, k, v, do, heads_per_pass, want_o_f32, partials=not fused,
                     kv_heads_per_bwd_pass=kv_heads_per_bwd_pass)
    if fused:
        ds.forward_fused()
    else:
        ds.forward()
    out = {}
    if do is not None:
        ds.backward()
    torch.cuda.synchronize()
    ds.check_status()
    out["o"] = bf16_dev_to_f64(ds.o)
    out["lse"] = ds.lse.cpu().numpy()
    if want_o_f32:
        out["o_f32"] = ds.o_f32.cpu().numpy()
    if keep_partials:
        out["o_partial"] = ds.o_part.cpu().numpy()
        out["lse_partial"] = ds.lse_part.cpu().numpy()
    if do is not None:
        out["dq"], out["dk"], out["dv"] = bf16_dev_to_f64(ds.dq), bf16_dev_to_f64(ds.dk), bf16_dev_to_f64(ds.dv)
    out["state"] = ds
    return out
