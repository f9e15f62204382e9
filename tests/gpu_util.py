"""Shared by the GPU tests: run the library on a workload and compare with the oracle."""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

import oracle
import paper_2510_02613_b200 as E
import workloads as W
from workloads import device as WD

KINDS = {E.PHASE_EXPERTS: W.KIND_EXPERTS, E.PHASE_ATTN: W.KIND_ATTN, E.PHASE_KV: W.KIND_KV}


def oracle_phase(wl, phase, src, dst):
    if phase == E.PHASE_EXPERTS:
        oracle.reshard_experts(wl.shape, wl.old.placement, wl.new.placement, src, dst,
                               fused_w13=wl.fused_w13)
    elif phase == E.PHASE_ATTN:
        oracle.reshard_attn(wl.shape, wl.old.tp, wl.new.tp, src, dst, fused_qkv=wl.fused_qkv,
                            replicas=wl.attn_replicas)
    else:
        oracle.reshard_kv(wl.shape, wl.old, wl.new, src, dst, head_major=wl.kv_head_major)


def make_plan(wl, **kw):
    """A plan with the workload's layout variants."""
    return E.Plan(wl.shape, wl.old, wl.new, fused_w13=wl.fused_w13,
                  kv_head_major=wl.kv_head_major, fused_qkv=wl.fused_qkv,
                  attn_replicas=wl.attn_replicas, **kw)


def run_phase(plan, phase, src, dst, stream=None):
    fn = {E.PHASE_EXPERTS: plan.reshard_experts, E.PHASE_ATTN: plan.reshard_attn,
          E.PHASE_KV: plan.reshard_kv}[phase]
    fn(src, dst, stream)


def check_phase_full(wl, plan, phase, src=None):
    """Whole arenas, byte for byte, including bytes the phase must not write."""
    so = plan.arena_bytes(phase, E.SIDE_OLD)
    sn = plan.arena_bytes(phase, E.SIDE_NEW)
    if src is None:
        src = WD.alloc_filled(so, wl.seed, KINDS[phase])
    dst = WD.alloc_const(sn)
    run_phase(plan, phase, src, dst)
    torch.cuda.synchronize()
    h_src = [t.cpu().numpy() for t in src]
    want = [np.full(n, WD.FILL_BYTE, np.uint8) for n in sn]
    oracle_phase(wl, phase, h_src, want)
    for r, (g, w) in enumerate(zip(dst, want)):
        g = g.cpu().numpy()
        if not np.array_equal(g, w):
            bad = np.flatnonzero(g != w)
            raise AssertionError("%s phase %d rank %d: %d bytes differ, first at %d"
                                 % (wl.name, phase, r, bad.size, bad[0]))
    assert plan.device_status() == 0
    return src, dst


def check_phase_layers(wl, plan, phase, src, dst, layers):
    """Full-size run already done into dst: compare the given layers with the oracle
    run on those layers alone (layers are independent in every phase).  A few layers are
    in flight at once: the oracle call and the comparisons release the interpreter lock."""
    from concurrent.futures import ThreadPoolExecutor
    L = wl.shape.n_layers
    wl1 = wl.with_layers(1)

    def one(l):
        h_src = []
        for t in src:
            per = t.numel() // L
            h_src.append(t[l * per:(l + 1) * per].cpu().numpy())
        want = [np.full(t.numel() // L, WD.FILL_BYTE, np.uint8) for t in dst]
        oracle_phase(wl1, phase, h_src, want)
        for r, (t, w) in enumerate(zip(dst, want)):
            per = t.numel() // L
            g = t[l * per:(l + 1) * per].cpu().numpy()
            if not np.array_equal(g, w):
                bad = np.flatnonzero(g != w)
                raise AssertionError("%s phase %d layer %d rank %d: %d bytes differ, first at %d"
                                     % (wl.name, phase, l, r, bad.size, bad[0]))

    with ThreadPoolExecutor(max_workers=4) as pool:
        for _ in pool.map(one, layers):
            pass


def check_step_full(wl, plan):
    """emoe_reshard_step: all three phases in one call, whole arenas against the oracle."""
    src, dst, want = [], [], []
    for phase in range(3):
        so, sn = plan.arena_bytes(phase, E.SIDE_OLD), plan.arena_bytes(phase, E.SIDE_NEW)
        src.append(WD.alloc_filled(so, wl.seed, KINDS[phase]))
        dst.append(WD.alloc_const(sn))
    plan.reshard_step(src, dst)
    torch.cuda.synchronize()
    for phase in range(3):
        w = [np.full(t.numel(), WD.FILL_BYTE, np.uint8) for t in dst[phase]]
        oracle_phase(wl, phase, [t.cpu().numpy() for t in src[phase]], w)
        for r, (g, x) in enumerate(zip(dst[phase], w)):
            g = g.cpu().numpy()
            if not np.array_equal(g, x):
                bad = np.flatnonzero(g != x)
                raise AssertionError("%s step, phase %d rank %d: %d bytes differ, first at %d"
                                     % (wl.name, phase, r, bad.size, bad[0]))
    assert plan.device_status() == 0
