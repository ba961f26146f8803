"""Time stamps of one cluster of the tensor-core decode kernel (decode_pair_kernel).

    python -m paper_2512_06727_b200.trace --workload c5 --batch 32 --layer 0 --cluster 0

builds the library with -DKVCAR_TC_TRACE (libkvcar_trace.so, beside the regular one), fills a cache of the
workload's shape with seeded random rows, runs kvcar_decode_attention on one layer three times and prints, from the
stamps of the last launch, what the chosen cluster's MMA issuer and first epilogue warp did: per accumulator job its
duration, the K slabs it walked, the time between a slab's release and the next slab's operands being seen ("wait")
and the time spent issuing ("issue"), and per job the epilogue's wait and work.  Clock: clock64 of the leader CTA's SM.
The stamps cost about 36 cycles each; the totals agree with an unstamped launch within a few per cent, but stamps
placed between individual asynchronous instructions lengthen what they measure (each then waits for its predecessor).
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import sys

import numpy as np


def main(argv=None) -> int:
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--workload", default="c5", choices=["c2", "c3", "c4", "c5"])
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--layer", type=int, default=0)
    ap.add_argument("--cluster", type=int, default=0)
    ap.add_argument("--jobs", type=int, default=14, help="jobs to list")
    ap.add_argument("--absorbed", action="store_true", help="pass KVCAR_ABSORBED")
    ap.add_argument("--absorbed-v", action="store_true", help="with --absorbed: KVCAR_ABSORBED_V as well")
    ap.add_argument("--json", default=None, help="also write the raw stamps here")
    args = ap.parse_args(argv)

    import torch
    from . import binding as B
    lib = B.load(trace=True)
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import kvcar_synth as synth
    from .session import Session

    w = synth.scaled(synth.CONFIGS[args.workload], batch=args.batch)
    src = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
    aes = synth.make_stack_autoencoders(w, src, src)
    pps = (w.cached_tokens + 2 + w.page_tokens - 1) // w.page_tokens
    sess = Session(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, w.batch, w.batch * pps, pps,
                   w.storage, src, src, aes)
    seqs = list(range(w.batch))
    for s in seqs:
        sess.ctx.seq_open(s)
    g = torch.Generator(device=sess.device)
    g.manual_seed(w.seed)
    kvw = w.n_kv_heads * w.head_dim
    chunk = 1024
    for t in range(0, w.cached_tokens, chunk):
        n = min(chunk, w.cached_tokens - t)
        for l in range(w.n_layers):
            k = torch.randn(w.batch, n, kvw, generator=g, device=sess.device).to(sess.dtype)
            v = torch.randn(w.batch, n, kvw, generator=g, device=sess.device).to(sess.dtype)
            sess.ctx.encode_append_tensor(l, seqs, n, k.data_ptr(), v.data_ptr(), sess.stream())
            torch.cuda.current_stream().synchronize()
        sess.ctx.advance(seqs, n, sess.stream())
    k = torch.randn(w.n_layers, w.batch, kvw, generator=g, device=sess.device).to(sess.dtype)
    v = torch.randn(w.n_layers, w.batch, kvw, generator=g, device=sess.device).to(sess.dtype)
    q = torch.randn(w.batch, w.n_q_heads, w.head_dim, generator=g, device=sess.device).to(sess.dtype)
    out = torch.empty_like(q)
    for l in range(w.n_layers):
        sess.ctx.encode_append(l, seqs, 1, k[l].data_ptr(), v[l].data_ptr(), sess.stream())
    assert lib.kvcar_debug_trace_select(C.c_int(args.cluster)) == 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        e0.record()
        sess.ctx.decode_attention(args.layer, seqs, q.data_ptr(), out.data_ptr(),
                                  B.INCLUDE_CURRENT_EXACT | (B.ABSORBED if args.absorbed else 0) |
                                  (B.ABSORBED_V if args.absorbed and args.absorbed_v else 0), sess.stream())
        e1.record()
        torch.cuda.synchronize()
    sess.ctx.sync_status(sess.stream())
    print(f"workload {w.name} batch {w.batch} layer {args.layer}: kvcar_decode_attention {1e3 * e0.elapsed_time(e1):.1f} us"
          f" (tile kernel + combine, stamps on)")
    buf = (C.c_ulonglong * (2 * 4 * 4096))()
    n = (C.c_int * 8)()
    assert lib.kvcar_debug_trace_dump(buf, n) == 0
    arr = np.frombuffer(buf, dtype=np.uint64).reshape(2, 4, 4096)
    ev = {f"{c}.{r}": [(int(x >> 8), int(x & 0xFF)) for x in arr[c, r, :n[c * 4 + r]]] for c in range(2) for r in range(4)}
    if args.json:
        json.dump(ev, open(args.json, "w"))
    report(ev, args.jobs)
    return 0


def ring_legs(ev):
    """The staging ring's round trip in the head-group phase, from the producers' and the issuer's stamps of the
    leader CTA: both producers stamp every slab once they are past its place (the one that loads it after the load
    is issued), the issuer stamps operands seen (0x30) and products + release issued (0x31).  Slab i of a head-group
    job re-uses the place of slab i - 3 (a ring of three places, as at the GPT-2 shape)."""
    iss = ev["0.2"]
    prod = [[t for t, g in ev[f"0.{r}"] if g in (2, 3)] for r in (0, 1)]
    seen, rel, kind = [], [], []
    k = None
    for t, tag in iss:
        if tag in (0x11, 0x12, 0x13, 0x14):
            k = tag & 7
        elif tag == 0x30:
            seen.append(t)
            kind.append(k)
        elif tag == 0x31:
            rel.append(t)
    n = min(len(seen), len(rel), len(prod[0]), len(prod[1]))
    if n < 8:
        return
    load, free, gap = [], [], []
    for i in range(n):
        if kind[i] != 2:
            continue
        issued = max(prod[0][i], prod[1][i])
        load.append(seen[i] - issued)
        if i + 3 < n and kind[i + 3] == 2:
            free.append(min(prod[0][i + 3], prod[1][i + 3]) - rel[i])
        if i > 0 and kind[i - 1] == 2:
            gap.append(seen[i] - rel[i - 1])
    if not load or not free:
        return
    med = lambda v: sorted(v)[len(v) // 2]
    print(f"  head-group ring: load issued -> operands seen by the issuer: median {med(load)} cycles; products + release issued"
          f" (slab i) -> place seen free for slab i+3: median {med(free)}; release issued -> next operands seen: median"
          f" {med(gap)}; issue of a slab (0x30 -> 0x31): median {med([r - s for r, s, k in zip(rel, seen, kind) if k == 2])}")


def report(ev, n_list):
    iss, ep = ev["0.2"], ev["0.3"]
    if not iss or not ep:
        print("no stamps: the chosen cluster does not exist in this launch, or the layer ran on another kernel")
        return
    t_zero = min(iss[0][0], ep[0][0])
    jobs, cur, last = [], None, None
    for t, tag in iss:
        if tag in (0x11, 0x12, 0x13, 0x14):
            cur = dict(kind=tag & 7, t0=t, wait=0, issue=0, slabs=0, prev=t)
            jobs.append(cur)
        elif tag == 0x30:
            cur["wait"] += t - cur["prev"]
            last = t
        elif tag == 0x31:
            cur["issue"] += t - last
            cur["slabs"] += 1
            cur["prev"] = t
        elif tag == 0x19:
            cur["t1"] = t
    ejobs, c = [], None
    for t, tag in ep:
        ph, kind = tag & 0xF, tag >> 4
        if ph == 0:
            c = dict(kind=kind, w0=t)
            ejobs.append(c)
        elif ph == 1:
            c["seen"] = t
        elif ph == 3:
            c["done"] = t
    names = {1: "hidden chunk", 2: "head group", 3: "K scores", 4: "V sums"}
    print("job  kind          start     cycles slabs   wait  issue | epilogue: job seen complete  work")
    for i, (j, e) in enumerate(zip(jobs, ejobs)):
        if i >= n_list or "t1" not in j or "done" not in e:
            break
        print(f"{i:3d}  {names[j['kind']]:12s} {j['t0'] - t_zero:8d} {j['t1'] - j['t0']:8d} {j['slabs']:5d} {j['wait']:6d} {j['issue']:6d} |"
              f" {e['seen'] - t_zero:10d} (+{e['seen'] - j['t1']:4d} after the commit) {e['done'] - e['seen']:6d}")
    done = [j for j in jobs if "t1" in j]
    span = iss[-1][0] - iss[0][0]
    print(f"issuer: {len(done)} jobs, {sum(j['slabs'] for j in done)} slabs in {span} cycles; waiting {sum(j['wait'] for j in done)},"
          f" issuing {sum(j['issue'] for j in done)}, between jobs {sum(done[i + 1]['t0'] - done[i]['t1'] for i in range(len(done) - 1))}")
    for kind in (1, 2, 3, 4):
        sel = [j for j in done if j["kind"] == kind]
        if sel:
            print(f"  {names[kind]} jobs: {len(sel)}, mean {sum(j['t1'] - j['t0'] for j in sel) / len(sel):.0f} cycles,"
                  f" {sum(j['t1'] - j['t0'] for j in sel) / max(1, sum(j['slabs'] for j in sel)):.0f} per slab")
    ring_legs(ev)
    for kind, nm in ((4, "hidden chunk"), (5, "K head group"), (6, "V head group")):
        sel = [e for e in ejobs if e["kind"] == kind and "done" in e and "seen" in e]
        if sel:
            print(f"  epilogue, {nm}: {len(sel)} jobs, mean wait {sum(e['seen'] - e['w0'] for e in sel) / len(sel):.0f},"
                  f" mean work {sum(e['done'] - e['seen'] for e in sel) / len(sel):.0f} cycles")


if __name__ == "__main__":
    sys.exit(main())
