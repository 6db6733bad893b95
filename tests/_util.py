"""Shared helpers of the GPU parity tests: moving seeded numpy inputs to the device and the
error measure of the parity bar (max |err| / max |ref| per output tensor)."""
import numpy as np

TOL_BF16 = 2e-2   # bf16 inputs, fp32 accumulation
TOL_F32 = 1e-4    # fp32 validation build


def torch_dtype(name):
    import torch
    return torch.bfloat16 if name == "bf16" else torch.float32


def dev(a, dtype_name="f32", device="cuda:0"):
    """numpy float32 (values already representable in the target dtype) -> CUDA tensor."""
    import torch
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if t.dtype == torch.float32:
        t = t.to(torch_dtype(dtype_name))
    return t.to(device)


def host(t):
    import torch
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def rel_err(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if ref.size == 0:
        return 0.0
    assert np.all(np.isfinite(got)), "non-finite values in the GPU result"
    return float(np.max(np.abs(got - ref)) / max(np.max(np.abs(ref)), 1e-30))


def prefill_to_device(p, device="cuda:0"):
    """PrefillInputs -> dict of CUDA tensors in the workload's dtype (s0 fp32, cu int32)."""
    import torch
    d = {name: dev(getattr(p, name), p.dtype, device) for name in ("q", "k", "x", "y", "v")}
    d["s0"] = None if p.s0 is None else torch.from_numpy(p.s0).to(device)
    d["cu"] = None if p.cu_seqlens is None else torch.from_numpy(p.cu_seqlens).to(device)
    d["cu_host"] = None if p.cu_seqlens is None else torch.from_numpy(p.cu_seqlens)
    return d
