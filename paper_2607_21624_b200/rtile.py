"""Offline tile selection for B200 (the paper's section 4.2 selection procedure and section 6 profiling step).

Two levels, as in the paper:

* storage tile (the R-Tile proper): ``candidates`` runs the library's progressive filter C1 -> C2 -> C3 over the
  initial pool and ranks the survivors by N_cache (Eq. 1) and padding;
* compute-tile configuration of each GEMM launch of the step (output-tile width, CTA-pair kernel, epilogue warp
  sets, and the slice count of the token-axis reductions): ``sweep`` is the hardware-profiling step (it times every
  legal configuration of every launch on the GPU at hand) and ``choose`` takes, per launch, the argmax of Eq. 2,
  sum over the launch's operators of GFLOPS x MemEfficiency, with MemEfficiency = minimal bytes / bytes the
  configuration's tiles fetch.  The result is a small JSON table keyed by layer shape, fixed before training and
  applied to a plan with ``apply`` (``LayerRunner`` does so when the table has the layer's shape).

    python -m paper_2607_21624_b200.rtile --configs 2 3 4 5 --out paper_2607_21624_b200/tuned_b200.json
"""
from __future__ import annotations

import ctypes as C
import itertools
import json
import os

from .binding import _check, lib

HERE = os.path.dirname(os.path.abspath(__file__))
DEFAULT_TABLE = os.path.join(HERE, "tuned_b200.json")
LAUNCHES = ["proj_qkv", "proj_o", "dWo+dA", "dWqkv+dXn"]          # FBL_GEMM_* ids in order


class RtileCand(C.Structure):
    _fields_ = [("tile_h", C.c_int32), ("tile_w", C.c_int32), ("n_cache", C.c_int32), ("pad_ratio", C.c_float)]


def candidates(shapes, elem_bytes=2, max_pad_ratio=0.10):
    """Storage-tile candidates for matrices of the given (rows, cols): list of dicts, best first, and the number of
    pool entries each constraint removed."""
    L = lib()
    L.fbl_rtile_candidates.argtypes = [C.POINTER(C.c_int64), C.c_int, C.c_int, C.c_float, C.POINTER(RtileCand), C.c_int,
                                       C.POINTER(C.c_int32)]
    flat = (C.c_int64 * (2 * len(shapes)))(*[int(v) for rc in shapes for v in rc])
    out = (RtileCand * 64)()
    rej = (C.c_int32 * 3)()
    n = L.fbl_rtile_candidates(flat, len(shapes), elem_bytes, max_pad_ratio, out, 64, rej)
    if n < 0:
        _check(n)
    cands = [dict(tile_h=out[i].tile_h, tile_w=out[i].tile_w, n_cache=out[i].n_cache, pad_ratio=out[i].pad_ratio)
             for i in range(min(n, 64))]
    return cands, dict(C1=rej[0], C2=rej[1], C3=rej[2])


def layer_matrix_shapes(cfg):
    n = cfg.seq                     # every sequence starts on a tile boundary, so each one is padded on its own
    return [(n, cfg.d_model), (n, cfg.d_q), (n, cfg.d_kv), (cfg.d_model, cfg.d_q), (cfg.d_model, cfg.d_kv), (cfg.d_q, cfg.d_model)]


def shape_key(cfg):
    return (f"B{cfg.batch}_T{cfg.seq}_D{cfg.d_model}_Hq{cfg.n_q_heads}_Hkv{cfg.n_kv_heads}_hd{cfg.head_dim}_"
            f"{cfg.dtype}_{'c' if cfg.causal else 'f'}_{'b' if cfg.has_bias else 'n'}")


def launch_ops(cfg):
    """Per launch: its operators as (M, N, K) products."""
    n, d, dq, dkv = cfg.batch * cfg.seq, cfg.d_model, cfg.d_q, cfg.d_kv
    return {"proj_qkv": [(n, dq, d), (n, dkv, d), (n, dkv, d)], "proj_o": [(n, d, dq)],
            "dWo+dA": [(dq, d, n), (n, dq, d)],
            "dWqkv+dXn": [(d, dq, n), (d, dkv, n), (d, dkv, n), (n, d, dq + 2 * dkv)]}


L2_RESIDENT_BYTES = 96e6           # of the 126 MB L2: a launch whose operands fit is re-read from L2, not from HBM


def mem_efficiency(ops, tile_m, tile_n, e=2, l2_bytes=L2_RESIDENT_BYTES):
    """Minimal bytes (each operand and the output once) over the bytes that cross HBM: once-only while the launch's
    operands stay L2-resident, else what the tiles of this shape fetch (every output tile reads its A rows and B
    columns over the whole reduction)."""
    minimal = fetched = 0.0
    for m, n, k in ops:
        tm, tn = -(-m // tile_m), -(-n // tile_n)
        minimal += (m * k + k * n + m * n) * e
        fetched += (tm * tn * (tile_m + tile_n) * k + m * n) * e
    return 1.0 if minimal <= l2_bytes else minimal / fetched


def legal_choices(cfg):
    """Every (tile_n, cta_pair, epilogue_sets) worth timing: 128- or 256-wide single-CTA tiles with one or two sets of
    epilogue warps, and the 256 x 256 CTA-pair tile."""
    out = [(bn, 0, es) for bn in (128, 256) for es in (1, 2)]
    out.append((256, 1, 1))
    return out


def apply(plan, choices):
    """choices: {launch name: [tile_n, cta_pair, epilogue_sets]}"""
    L = lib()
    L.fbl_plan_set_gemm_choice.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int]
    for name, (bn, pair, es) in choices.items():
        _check(L.fbl_plan_set_gemm_choice(plan._h, LAUNCHES.index(name), int(bn), int(pair), int(es)))


def load_table(path=None):
    path = path or DEFAULT_TABLE
    if not os.path.exists(path):
        return {}
    with open(path) as f:
        return json.load(f)


def sweep(cfg, reps=5, ksplits=((0, 0),)):
    """The profiling step: times each launch under each configuration (per-step device events of the library), L2
    flushed before every pass.  Returns {launch: {choice: ms}} per (ksplit_o, ksplit_qkv) setting (0 = the plan's own)."""
    import torch

    from fbl_inputs import make_inputs

    from .binding import LayerRunner
    inp = make_inputs(cfg)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    results = {}
    for ks_o, ks_qkv in ksplits:
        for k, v in (("FBL_KSPLIT_O", ks_o), ("FBL_KSPLIT_QKV", ks_qkv)):
            if v:
                os.environ[k] = str(v)
            else:
                os.environ.pop(k, None)
        run = LayerRunner(cfg, tile_choices={})
        run.load_inputs(inp)
        run.step()
        assert run.status() == 0
        times = {name: {} for name in LAUNCHES}
        for choice in legal_choices(cfg):
            apply(run.plan, {name: choice for name in LAUNCHES})
            run.step()                                   # sets kernel attributes of variants not used before
            run.plan.profile_enable(True)
            acc = {}
            for _ in range(reps):
                flush.zero_()
                run.forward()
                torch.cuda.synchronize()
                for name, t in run.plan.profile_read():
                    acc.setdefault(name, []).append(t)
                run.backward()
                torch.cuda.synchronize()
                for name, t in run.plan.profile_read():
                    acc.setdefault(name, []).append(t)
            run.plan.profile_enable(False)
            assert run.status() == 0
            for name in LAUNCHES:
                if name in acc:
                    times[name][choice] = min(acc[name])
        results[(ks_o, ks_qkv)] = times
        del run
        for k in ("FBL_KSPLIT_O", "FBL_KSPLIT_QKV"):
            os.environ.pop(k, None)
    return results


def choose(cfg, times):
    """Eq. 2 per launch: argmax over configurations of sum_ops GFLOPS x MemEfficiency.  All operators of a launch share
    its measured time, so the sum reduces to (launch GFLOPS) x (MemEfficiency over the launch's operators)."""
    ops = launch_ops(cfg)
    picked, table = {}, {}
    for name, per_choice in times.items():
        flops = sum(2.0 * m * n * k for m, n, k in ops[name])
        best, best_score = None, -1.0
        for (bn, pair, es), ms in per_choice.items():
            tile_m = 256 if pair else 128
            score = flops / (ms * 1e-3) / 1e9 * mem_efficiency(ops[name], tile_m, bn)
            table[f"{name}|{bn},{pair},{es}"] = dict(ms=ms, gflops=flops / (ms * 1e-3) / 1e9,
                                                     mem_eff=mem_efficiency(ops[name], tile_m, bn), score=score)
            if score > best_score:
                best, best_score = (bn, pair, es), score
        if best is not None:
            picked[name] = list(best)
    return picked, table


def main():
    import argparse

    from fbl_inputs import get_config
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", type=int, nargs="+", default=[2, 3, 4, 5])
    ap.add_argument("--out", default=DEFAULT_TABLE)
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--fastest", action="store_true", help="rank by measured time alone instead of Eq. 2's product")
    args = ap.parse_args()
    table = load_table(args.out)
    for i in args.configs:
        cfg = get_config(i)
        cands, rej = candidates(layer_matrix_shapes(cfg), 2 if cfg.dtype == "bf16" else 4)
        print(f"{cfg.name}: storage-tile candidates {cands[:3]} (removed by C1/C2/C3: {rej})")
        if cfg.dtype != "bf16":
            continue
        res = sweep(cfg, reps=args.reps)[(0, 0)]
        picked, detail = choose(cfg, res)
        if args.fastest:
            picked = {name: list(min(pc, key=pc.get)) for name, pc in res.items() if pc}
        for name in LAUNCHES:
            row = {f"{c[0]},{c[1]},{c[2]}": round(ms * 1e3, 1) for c, ms in sorted(res[name].items())}
            print(f"  {name:10s} us by (tile_n,pair,esets): {row} -> {picked.get(name)}")
        table[shape_key(cfg)] = {"choices": picked, "workload": cfg.name}
    with open(args.out, "w") as f:
        json.dump(table, f, indent=1, sort_keys=True)
    print("wrote", args.out)


if __name__ == "__main__":
    main()
