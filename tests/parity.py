"""Comparators and drivers shared by the GPU parity tests."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

import oracle
import synth

MOM = float(np.float32(0.9))     # the library keeps momentum in fp32; give the oracle the same number
LR = float(np.float32(0.1))


def max_rel_err(a, b, floor=1e-2):
    """max |a-b| / max(|b|, floor*max|b|): relative error, with elements below 1 % of the tensor's largest
    magnitude compared against that 1 % instead.  An fp32 chain of k roundings leaves an absolute error of
    about k * 6e-8 * scale on every element whatever its own size (the error follows the summands, not the
    sum), so a 1e-4 relative bound is only meaningful for elements above k * 6e-4 of the scale; k ~ 10."""
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    s = np.abs(b).max()
    if s == 0:
        return float(np.abs(a).max())
    return float((np.abs(a - b) / np.maximum(np.abs(b), floor * s)).max())


def norm_max_abs(a, b):
    """max|a-b| / max|b| (the bf16 criterion)."""
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    s = np.abs(b).max()
    return float(np.abs(a - b).max() / s) if s > 0 else float(np.abs(a).max())


def per_tensor(arch, a, b, fn, skip_blocks=(), skip_names=()):
    """Worst fn(a_t, b_t) over the parameter tensors; returns (value, tensor name)."""
    worst, name = 0.0, ""
    for t in synth.param_layout(arch)[0]:
        if t.block in skip_blocks or t.name in skip_names:
            continue
        v = fn(a[t.offset:t.offset + t.size], b[t.offset:t.offset + t.size])
        if v > worst:
            worst, name = v, t.name
    return worst, name


def to_dev(x, dtype):
    t = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    return t.to(dtype) if t.dtype.is_floating_point else t


def run_protocol_both(arch, S, B, steps, seed, dtype, quant, grouped, lib_mod, policy_seed=77, lr=LR, mu=MOM,
                      conv_backend=0, with_oracle=True):
    """One ResIST round on both sides from identical inputs.  Returns a dict of everything comparable."""
    a = arch.to_int32()
    p0, buf0 = synth.perturbed_params(arch, seed)
    ctx = lib_mod.Context(a, dtype=lib_mod.BF16 if dtype == "bf16" else lib_mod.F32, momentum=mu, conv_backend=conv_backend)
    ctx.set_params(p0, buf0)
    mask_gpu = ctx.partition(policy_seed, S)
    mask_cpu = oracle.partition(a, policy_seed, S)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    out = {"mask_gpu": mask_gpu, "mask_cpu": mask_cpu, "steps": [], "arch": arch}
    subs = [p0.copy() for _ in range(S)]
    moms = [np.zeros_like(p0) for _ in range(S)]
    bufs = [buf0.copy() for _ in range(S)]
    n_img = arch.in_h * arch.in_w * arch.in_c
    for step in range(steps):
        xs, ys = [], []
        for s in range(S):
            x = synth.standard_normal(seed * 1000 + step * 37 + s, B * n_img).astype(np.float32).reshape(B, arch.in_h, arch.in_w, arch.in_c)
            if dtype == "bf16":
                x = synth.round_to_bf16(x)
            y = (synth.splitmix64_words(seed * 77 + step * 5 + s, B) % np.uint64(arch.classes)).astype(np.int32)
            xs.append(x)
            ys.append(y)
        dx = [to_dev(x, tdt) for x in xs]
        dy = [to_dev(y, None) for y in ys]
        loss = torch.zeros(S, dtype=torch.float32, device="cuda")
        if grouped:
            ctx.local_step_grouped(dx, dy, lr, loss)
        else:
            for s in range(S):
                ctx.local_step(s, dx[s], dy[s], lr, loss[s:s + 1])
        torch.cuda.synchronize()
        rec = {"loss_gpu": loss.cpu().numpy(), "subs": []}
        # the sub-ResNets are independent: the oracle steps them on one host thread each (the C routine releases the interpreter)
        if not with_oracle:                   # GPU side only (a second backend on inputs the oracle has already seen)
            rec["subs"] = [{"logits_gpu": ctx.get_logits(s, B), "grads_gpu": ctx.get_grads(s)} for s in range(S)]
            out["steps"].append(rec)
            continue
        with ThreadPoolExecutor(max_workers=max(1, min(S, os.cpu_count() or 1))) as ex:
            outs = list(ex.map(lambda s: oracle.step(a, oracle.present_of(mask_cpu, s), subs[s], moms[s], bufs[s], xs[s], ys[s], lr=lr, mu=mu,
                                                     quant=quant), range(S)))
        for s in range(S):
            o = outs[s]
            gp, gb = ctx.get_params(s)
            rec["subs"].append({"loss_cpu": o["loss"], "logits_cpu": o["logits"], "grads_cpu": o["grads"],
                                "params_cpu": subs[s].copy(), "bufs_cpu": bufs[s].copy(),
                                "logits_gpu": ctx.get_logits(s, B), "grads_gpu": ctx.get_grads(s), "params_gpu": gp, "bufs_gpu": gb})
        out["steps"].append(rec)
    out.update(ctx=ctx, info=ctx.step_info())
    if not with_oracle:
        return out
    # reassembly: the oracle applied to the GPU's own working copies must match bit for bit
    gsubs = [ctx.get_params(s) for s in range(S)]
    ctx.aggregate()
    gp, gb = ctx.get_params(-1)
    ref_p, ref_b = p0.copy(), buf0.copy()
    oracle.aggregate(a, mask_cpu, [g[0] for g in gsubs], [g[1] for g in gsubs], ref_p, ref_b)
    out.update(global_gpu=gp, global_buf_gpu=gb, global_from_gpu_subs=ref_p, global_buf_from_gpu_subs=ref_b)
    e2e_p, e2e_b = p0.copy(), buf0.copy()
    oracle.aggregate(a, mask_cpu, subs, bufs, e2e_p, e2e_b)
    out.update(global_cpu=e2e_p, global_buf_cpu=e2e_b, ctx=ctx, info=ctx.step_info())
    return out
