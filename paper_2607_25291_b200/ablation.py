"""Remapping analysis and kernel microbenchmark on synthetic workloads (needs a B200).

Two tables, both produced with the library's own kernels only:

* ``remap``  (Sec. 5.3 "Effect of remapping"; Sec. D "Full Remapping Sweep"): the same Stage-1 sets are
  visited in KAP order ("with remapping") and in natural page order ("without"), for Stage-1 budgets
  {100, 54, 42, 32, 28} % and a sweep of the skip scale Delta.  Reported: the in-kernel skip ratio
  (1 - computed / listed) and, standing in for perplexity (no model here), the relative L2 error of the
  output against the Stage-1-only output (Delta = -1).
* ``micro``  (Sec. D "Kernel Microbenchmark"): index-driven jumping over the order lists against a
  logical-mask walk of the same sets (``cosa_options.logical_mask``), Stage 2 off, at budgets
  {25, 50, 75} % and 32K / 64K / 128K, with the library's dense path and PyTorch SDPA as the dense
  references.

* ``sweep``  the 64K budget sweep: Stage-1 {50, 25, 12.5} % x Stage-2 {off, 0.5x, 0.25x}: latencies, blocks listed /
  scored / computed, distance of the output from dense attention.
* ``stack``  the 36-layer stack of 128K layers with layer-varying needle density: attention time of the whole
  prefill (KAP + OSK per layer, summed) against the library's dense path and PyTorch SDPA.

    python -m paper_2607_25291_b200.ablation remap [--workload qwen3_32k]
    python -m paper_2607_25291_b200.ablation micro [--lengths 32k,64k,128k]
    python -m paper_2607_25291_b200.ablation stack [--workload qwen3_128k_x36] [--dense-every 6]
    python -m paper_2607_25291_b200.ablation sweep        (the 64K budget sweep)
"""
import argparse
import json
import os

import numpy as np
import torch

from . import binding as cosa

REMAP_BUDGETS = (1.0, 0.54, 0.42, 0.32, 0.28)
MICRO_BUDGETS = (0.25, 0.5, 0.75)
MICRO_WORKLOADS = {"32k": "qwen3_32k", "64k": "llama31_64k_sweep", "128k": "qwen3_128k"}


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()[None].contiguous()


def _time(fn, reps=3):
    fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    if cosa.cosa_device_status() != 0:
        raise RuntimeError("device status reports a timed-out wait")
    return a.elapsed_time(b) / reps


class Problem:
    """Device tensors of one synthetic layer and the buffers the calls write."""

    def __init__(self, workload):
        self.w = workload
        qb, kb, vb, _ = workload.make()
        self.q, self.k, self.v = _dev(qb), _dev(kb), _dev(vb)
        self.nqb = workload.n_blocks
        hq = workload.hq
        self.shape = cosa.make_shape(self.q, self.k, True)
        self.order = torch.empty(1, hq, self.nqb, self.nqb, dtype=torch.int32, device="cuda")
        self.count = torch.empty(1, hq, self.nqb, dtype=torch.int32, device="cuda")
        self.out = torch.empty_like(self.q)
        self.visited = torch.empty(1, hq, self.nqb, dtype=torch.int32, device="cuda")

    def select(self, budget):
        cosa.cosa_kap_select(self.q, self.k, budget, self.order, self.count,
                             opt=cosa.default_options(stride=self.w.stride, order_stride=self.nqb))

    def attend(self, order, skip_scale, tightened_budget, out=None, mask=None):
        opt = cosa.default_options(skip_scale=skip_scale, order_stride=self.nqb, logical_mask=mask)
        cosa.cosa_osk_attention(self.q, self.k, self.v, order, None if mask is not None else self.count,
                                tightened_budget, self.out if out is None else out, None, self.visited, opt=opt)


def remap_table(workload, budgets=REMAP_BUDGETS, deltas=None):
    """Rows of (stage-1 budget, Delta, skip ratio with / without remapping, relative error with / without)."""
    pb = Problem(workload)
    if deltas is None:
        base = workload.skip_scale
        deltas = [min(base * f, 0.9 * workload.n) for f in (0.0625, 0.125, 0.25, 0.5, 1.0)]
    rows = []
    ref = torch.empty_like(pb.q)
    natural = torch.empty_like(pb.order)
    got = torch.empty_like(pb.q)
    for b1 in budgets:
        pb.select(b1)
        natural.copy_(pb.order)
        cosa.cosa_reorder_lists(natural, pb.count, pb.shape)
        listed = int(pb.count.sum())
        pb.attend(pb.order, -1.0, 1.0, out=ref)                     # Stage 1 only: no in-kernel skipping
        ref_norm = float(ref.float().norm())
        for delta in deltas:
            cell = []
            for order in (pb.order, natural):
                pb.attend(order, float(delta), 0.99999, out=got)    # threshold on, cap not binding
                torch.cuda.synchronize()
                skip = 1.0 - int(pb.visited.sum()) / listed
                err = float((got.float() - ref.float()).norm()) / ref_norm
                cell.append((skip, err))
            rows.append(dict(stage1=b1, delta=float(delta), skip_remap=cell[0][0], skip_natural=cell[1][0],
                             err_remap=cell[0][1], err_natural=cell[1][1], listed=listed))
    if cosa.cosa_device_status() != 0:
        raise RuntimeError("device status reports a timed-out wait")
    return rows


def micro_table(workloads, budgets=MICRO_BUDGETS, with_sdpa=True):
    """Rows of (length, budget, ms: jump in KAP order / jump in natural order / logical-mask walk / dense path / SDPA)."""
    rows = []
    for w in workloads:
        pb = Problem(w)
        nqb, hq = pb.nqb, w.hq
        tri = torch.arange(nqb, device="cuda", dtype=torch.int32)
        full = torch.where(tri[None, :] <= tri[:, None], tri[None, :].expand(nqb, nqb),
                           torch.full((), -1, dtype=torch.int32, device="cuda")).expand(1, hq, nqb, nqb).contiguous()
        keep_order, keep_count = pb.order, pb.count
        pb.order, pb.count = full, (tri + 1).expand(1, hq, nqb).contiguous()
        dense_ms = _time(lambda: pb.attend(pb.order, -1.0, 1.0), reps=2)
        pb.order, pb.count = keep_order, keep_count
        del full
        sdpa_ms = None
        if with_sdpa:
            sdpa_ms = _time(lambda: torch.nn.functional.scaled_dot_product_attention(pb.q, pb.k, pb.v, is_causal=True,
                                                                                     enable_gqa=True), reps=2)
        natural = torch.empty_like(pb.order)
        mask = torch.empty(1, hq, nqb, (nqb + 31) // 32, dtype=torch.int32, device="cuda")
        for b in budgets:
            pb.select(b)
            natural.copy_(pb.order)
            cosa.cosa_reorder_lists(natural, pb.count, pb.shape)
            cosa.cosa_lists_to_mask(pb.order, pb.count, pb.shape, mask)
            jump = _time(lambda: pb.attend(pb.order, -1.0, 1.0))
            jump_nat = _time(lambda: pb.attend(natural, -1.0, 1.0))
            logical = _time(lambda: pb.attend(None, -1.0, 1.0, mask=mask))
            rows.append(dict(n=w.n, budget=b, listed=int(pb.count.sum()), jump_ms=jump, jump_natural_ms=jump_nat,
                             logical_ms=logical, dense_ms=dense_ms, sdpa_ms=sdpa_ms))
        del pb, natural, mask
        torch.cuda.empty_cache()
    return rows


class Journal:
    """Rows of a long table kept as JSON lines, so that a run that was cut short resumes where it stopped: rows already
    in the file are returned by `get` and not measured again."""

    def __init__(self, path):
        self.path, self.rows = path, {}
        if path and os.path.exists(path):
            with open(path) as f:
                for line in f:
                    line = line.strip()
                    if line:
                        row = json.loads(line)
                        self.rows[row["key"]] = row

    def get(self, key):
        return self.rows.get(key)

    def put(self, key, row):
        row = dict(row, key=key)
        self.rows[key] = row
        if self.path:
            with open(self.path, "a") as f:
                f.write(json.dumps(row) + "\n")
        return row


def stack_table(workload, dense_every=6, journal=None):
    """One row per layer: KAP ms, OSK ms, blocks computed; the dense references are timed on every dense_every-th
    layer (their time does not depend on the data) and averaged.  With a journal, layers it already holds are not run."""
    journal = journal or Journal(None)
    rows, dense_ms, sdpa_ms = [], [], []
    nqb, hq = workload.n_blocks, workload.hq
    pitch = (cosa.cosa_budget_count(workload.kap_budget, nqb) + 7) // 8 * 8
    order = torch.empty(1, hq, nqb, pitch, dtype=torch.int32, device="cuda")
    count = torch.empty(1, hq, nqb, dtype=torch.int32, device="cuda")
    visited = torch.empty(1, hq, nqb, dtype=torch.int32, device="cuda")
    opt = cosa.default_options(stride=workload.stride, skip_scale=workload.skip_scale, order_stride=pitch)
    out = None
    for layer in range(workload.layers):
        need_dense = layer % dense_every == 0
        have = journal.get(f"{workload.name}/layer{layer}")
        have_dense = journal.get(f"{workload.name}/dense{layer}") if need_dense else None
        if have is not None and (not need_dense or have_dense is not None):
            rows.append(have)
            if need_dense:
                dense_ms.append(have_dense["dense_ms"]); sdpa_ms.append(have_dense["sdpa_ms"])
            continue
        qb, kb, vb, _ = workload.make(layer=layer)
        q, k, v = _dev(qb), _dev(kb), _dev(vb)
        if out is None:
            out = torch.empty_like(q)
        kap = _time(lambda: cosa.cosa_kap_select(q, k, workload.kap_budget, order, count, opt=opt), reps=2)
        osk = _time(lambda: cosa.cosa_osk_attention(q, k, v, order, count, workload.osk_budget, out, None, visited, opt=opt), reps=2)
        rows.append(journal.put(f"{workload.name}/layer{layer}",
                                dict(layer=layer, kap_ms=kap, osk_ms=osk, listed=int(count.sum()), computed=int(visited.sum()))))
        if need_dense:
            tri = torch.arange(nqb, device="cuda", dtype=torch.int32)
            full = torch.where(tri[None, :] <= tri[:, None], tri[None, :].expand(nqb, nqb),
                               torch.full((), -1, dtype=torch.int32, device="cuda")).expand(1, hq, nqb, nqb).contiguous()
            fcount = (tri + 1).expand(1, hq, nqb).contiguous()
            dopt = cosa.default_options(order_stride=nqb)
            dense_ms.append(_time(lambda: cosa.cosa_osk_attention(q, k, v, full, fcount, 1.0, out, None, None, opt=dopt), reps=1))
            sdpa_ms.append(_time(lambda: torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True, enable_gqa=True), reps=1))
            journal.put(f"{workload.name}/dense{layer}", dict(dense_ms=dense_ms[-1], sdpa_ms=sdpa_ms[-1]))
            del full
        del q, k, v
    return rows, float(np.mean(dense_ms)), float(np.mean(sdpa_ms))


def _print_stack(rows, dense_ms, sdpa_ms):
    print("| layer | KAP ms | OSK ms | KAP+OSK ms | blocks listed | blocks computed |")
    print("|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['layer']} | {r['kap_ms']:.2f} | {r['osk_ms']:.2f} | {r['kap_ms'] + r['osk_ms']:.2f} | {r['listed']} | {r['computed']} |")
    total = sum(r["kap_ms"] + r["osk_ms"] for r in rows)
    n = len(rows)
    print(f"\ntotal over {n} layers: {total:.1f} ms; dense path {dense_ms:.1f} ms/layer = {dense_ms * n:.0f} ms "
          f"({dense_ms * n / total:.2f}x); SDPA {sdpa_ms:.1f} ms/layer = {sdpa_ms * n:.0f} ms ({sdpa_ms * n / total:.2f}x)")


def sweep_table(workload, stage1, stage2_mult):
    """The budget sweep: Stage-1 budget x (Stage-2 budget as a multiple of it; 1.0 = Stage 2 off): latencies, blocks
    listed / scored / computed, and the relative L2 distance of the output from the library's dense path."""
    pb = Problem(workload)
    nqb, hq = pb.nqb, workload.hq
    tri = torch.arange(nqb, device="cuda", dtype=torch.int32)
    full = torch.where(tri[None, :] <= tri[:, None], tri[None, :].expand(nqb, nqb),
                       torch.full((), -1, dtype=torch.int32, device="cuda")).expand(1, hq, nqb, nqb).contiguous()
    dense = torch.empty_like(pb.q)
    cosa.cosa_osk_attention(pb.q, pb.k, pb.v, full, (tri + 1).expand(1, hq, nqb).contiguous(), 1.0, dense, None, None,
                            opt=cosa.default_options(order_stride=nqb))
    del full
    dense_norm = float(dense.float().norm())
    scored = torch.empty_like(pb.visited)
    rows = []
    for b1 in stage1:
        kap = _time(lambda: pb.select(b1))
        for mult in stage2_mult:
            tb = 1.0 if mult == 1.0 else b1 * mult
            opt = cosa.default_options(skip_scale=workload.skip_scale, order_stride=nqb, out_scored=scored)
            osk = _time(lambda: cosa.cosa_osk_attention(pb.q, pb.k, pb.v, pb.order, pb.count, tb, pb.out, None, pb.visited, opt=opt))
            err = float((pb.out.float() - dense.float()).norm()) / dense_norm
            rows.append(dict(stage1=b1, stage2=tb, kap_ms=kap, osk_ms=osk, listed=int(pb.count.sum()), scored=int(scored.sum()),
                             computed=int(pb.visited.sum()), err=err))
    return rows


def _print_sweep(rows):
    print("| stage-1 budget | stage-2 budget | KAP ms | OSK ms | blocks listed | scored | computed | rel. L2 distance from dense |")
    print("|---|---|---|---|---|---|---|---|")
    for r in rows:
        s2 = "off" if r["stage2"] >= 1.0 else f"{r['stage2']:.4f}"
        print(f"| {r['stage1']:.3f} | {s2} | {r['kap_ms']:.2f} | {r['osk_ms']:.2f} | {r['listed']} | {r['scored']} | {r['computed']} | {r['err']:.3e} |")


def _print_remap(rows):
    print("| stage-1 budget | Delta | skip ratio, KAP order | skip ratio, natural order | rel. error, KAP order | rel. error, natural order |")
    print("|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['stage1']:.2f} | {r['delta']:.0f} | {r['skip_remap']:.3f} | {r['skip_natural']:.3f} | "
              f"{r['err_remap']:.2e} | {r['err_natural']:.2e} |")


def _print_micro(rows):
    print("| N | budget | jump, KAP order ms | jump, natural order ms | logical-mask walk ms | dense path ms | SDPA ms | "
          "speed-up of jump over SDPA | logical / jump (natural) |")
    print("|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        sd = r["sdpa_ms"]
        print(f"| {r['n']} | {r['budget']:.2f} | {r['jump_ms']:.3f} | {r['jump_natural_ms']:.3f} | {r['logical_ms']:.3f} | "
              f"{r['dense_ms']:.2f} | {sd if sd is None else round(sd, 2)} | "
              f"{'-' if sd is None else round(sd / r['jump_ms'], 2)} | {r['logical_ms'] / r['jump_natural_ms']:.3f} |")


def main():
    from synth.configs import WORKLOADS
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("table", choices=["remap", "micro", "stack", "sweep"])
    ap.add_argument("--dense-every", type=int, default=6)
    ap.add_argument("--workload", default="qwen3_32k")
    ap.add_argument("--lengths", default="32k,64k,128k")
    ap.add_argument("--jsonl", default=None,
                    help="stack: keep the per-layer rows in this file (JSON lines) and resume from it if it exists")
    args = ap.parse_args()
    if args.table == "sweep":
        from synth.configs import SWEEP_STAGE1, SWEEP_STAGE2_MULT
        _print_sweep(sweep_table(WORKLOADS["llama31_64k_sweep"], SWEEP_STAGE1, SWEEP_STAGE2_MULT))
    elif args.table == "stack":
        wl = WORKLOADS[args.workload if args.workload != "qwen3_32k" else "qwen3_128k_x36"]
        _print_stack(*stack_table(wl, args.dense_every, Journal(args.jsonl)))
    elif args.table == "remap":
        _print_remap(remap_table(WORKLOADS[args.workload]))
    else:
        _print_micro(micro_table([WORKLOADS[MICRO_WORKLOADS[x]] for x in args.lengths.split(",")]))


if __name__ == "__main__":
    main()
