"""Host glue shared by the tests and the benchmark: upload planes, build handles,
run the staged calls.  No arithmetic of the serving path lives here."""
import numpy as np
import torch

from . import binding as sf


def dev(a, device="cuda:0"):
    """numpy array -> device tensor with the same bytes (uint16/uint32 included)."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def upload_packets(pk, n_valid=None, device="cuda:0", with_hdr=True):
    t = {k: dev(pk[k], device) for k in ("size", "iat_us", "dir_bits")}
    t["hdr"] = dev(pk["hdr"], device) if (with_hdr and "hdr" in pk and pk["hdr"].shape[-1] > 0) else None
    t["n_valid"] = dev(np.asarray(n_valid, np.uint8), device) if n_valid is not None else None
    t["struct"] = sf.make_packets(t["size"], t["iat_us"], t["dir_bits"], t["hdr"], t["n_valid"])
    return t


def pinned_packets(pk, with_hdr=True, pinned=True):
    """Host copies for the host-pointer entry point: pinned (the device can address them: the assigned
    rows are pulled straight out of them) or pageable (staged through the library's own pinned buffer)."""
    t = {}
    for k in ("size", "iat_us", "dir_bits") + (("hdr",) if with_hdr else ()):
        t[k] = torch.from_numpy(np.ascontiguousarray(pk[k]).copy())
        if pinned:
            t[k] = t[k].pin_memory()
    hdr = t.get("hdr")
    t["struct"] = sf.make_packets(t["size"], t["iat_us"], t["dir_bits"], hdr, None)
    return t


def make_forest(ctx, fo):
    kind = {"rf": sf.SF_RF, "gbdt": sf.SF_GBDT, "gbdt_mc": sf.SF_GBDT_MC}[fo["kind"]]
    return sf.sf_forest_create(ctx, kind, fo["T"], fo["depth"], fo["F"], fo["C"], fo["fid"], fo["thr"], fo["leaf"])


def make_slow(ctx, cfg, model):
    dt = sf.SF_BF16 if cfg.slow_dtype == "bf16" else sf.SF_F32
    if cfg.slow == "mlp":
        return sf.sf_mlp_create(ctx, dt, model["dims"], model["W"], model["b"])
    return sf.sf_cnn_create(ctx, dt, model)


def bf16_bits_to_f32(t):
    """uint16/bf16 device tensor -> float32 numpy (exact)."""
    if t.dtype != torch.bfloat16:
        t = t.view(torch.bfloat16)
    return t.float().cpu().numpy()


def route_cfg_for(cfg, tau_dev, capacity, P_real=0):
    rule = sf.SF_LC_GT if cfg.kind == "rf" else sf.SF_ABSMARGIN_LT
    layout = sf.SF_MLP16 if cfg.slow == "mlp" else sf.SF_CNN8
    dt = sf.SF_BF16 if cfg.slow_dtype == "bf16" else sf.SF_F32
    return sf.make_route_cfg(rule, tau_dev, layout, dt, cfg.P, capacity, P_real)


class _DevPtr:
    def __init__(self, ptr, n, typestr):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (int(ptr), False), "version": 2}


def ptr_tensor(ptr, shape, dtype, device="cuda:0"):
    """Copy of library-owned device memory as a torch tensor (for inspection)."""
    n = int(np.prod(shape))
    esz = torch.empty(0, dtype=dtype).element_size()
    if n == 0:
        return torch.empty(shape, dtype=dtype, device=device)
    raw = torch.as_tensor(_DevPtr(ptr, n * esz, "|u1"), device=device)
    return raw.clone().view(dtype).view(*shape)
