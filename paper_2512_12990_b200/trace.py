"""Where the time of a decode launch goes: runs the DeepSeek-V2-Lite-shaped layer back to back through a library
built with the decode kernel's time stamps (-DSLICEMOE_TRACE) and prints, for the last launch, when each role of
the 148 CTAs passed its points - microseconds after the CTA's own dependency wait returned.

    python -m paper_2512_12990_b200.trace [dsv2|qwen] [--resident] [--per-cta]

Needs a CUDA device.  Builds paper_2512_12990_b200/libslicemoe_trace.so on first use; the ordinary library and
its timings are not affected (the stamped kernel is about 0.4 us per launch slower)."""
from __future__ import annotations

import ctypes
import sys
from ctypes import c_void_p

import numpy as np

NAMES = {1: "dependency wait over", 2: "plan built (warp 0)", 3: "x as digits (warp 3)", 4: "prologue barrier passed",
         5: "gate/up phase done, group 0", 6: "gate/up phase done, group 1", 7: "gate/up phase done, group 2",
         8: "gate/up phase done, group 3", 12: "last h value written", 9: "list of down chunks built (warp 0)",
         10: "own h blocks in digits (warp 0)", 11: "down phase done (warp 0)", 13: "y written"}
NAMES[31] = "producer 0 begins the down tiles"
NAMES[18] = "producer 0 has requested all down tiles"
NAMES[19] = "producer 1 has requested all down tiles"
for _j in range(8):
    NAMES[32 + _j] = f"producer 0 requests gate/up chunk {_j}"
for _j in range(4):
    NAMES[40 + _j] = f"producer 0: down chunk landed, #{_j} it waits for"
    NAMES[44 + _j] = f"producer 1: down chunk landed, #{_j} it waits for"
for _g in range(4):
    NAMES[14 + _g] = f"own h blocks in digits, group {_g}"
    NAMES[23 + _g] = f"last down chunk's h flagged, group {_g}"
    NAMES[27 + _g] = f"down phase done, group {_g}"


def main(argv):
    import torch
    from . import binding as B
    from . import build as builder
    from . import synth
    B._LIB_PATH = builder.build(trace=True)
    name = next((a for a in argv if a in ("dsv2", "qwen")), "dsv2")
    flags = B.LISTS_RESIDENT if "--resident" in argv else 0
    sh = synth.SHAPES[name]
    rank_high = 3 if name == "dsv2" else 2
    dev = torch.device("cuda", 0)
    L, P = 8, 64
    gen = torch.Generator(device=dev)
    gen.manual_seed(1)
    cs = B.make_shape(sh.hidden, sh.inter, sh.n_experts, sh.top_k, sh.group, sh.n_shared, sh.shared_inter,
                      sh.shared_sigmoid_gate)

    def pack3(n, k_):
        W = torch.empty((n, k_), dtype=torch.float32, device=dev)
        out = {}
        for key, shape_ in (("gate", (n, k_)), ("up", (n, k_)), ("down", (k_, n))):
            W = torch.empty(shape_, dtype=torch.float32, device=dev).normal_(0.0, 0.02, generator=gen)
            out[key] = B.slicemoe_pack(W, sh.group)
        return out

    keep, tables, shared_tables, gate_vecs = [], [], [], []
    for _ in range(L):
        ex = [pack3(sh.inter, sh.hidden) for _ in range(sh.n_experts)]
        shd = [pack3(sh.shared_inter, sh.hidden) for _ in range(sh.n_shared)]
        keep.append((ex, shd))
        tables.append(B.expert_table(ex, dev))
        shared_tables.append(B.expert_table(shd, dev) if shd else None)
        gate_vecs.append(torch.empty(sh.hidden, dtype=torch.float32, device=dev).normal_(0.0, 0.02, generator=gen)
                         if sh.shared_sigmoid_gate else None)
    ws = B.new_workspace(cs, dev)
    logits = torch.from_numpy(synth.router_logits_normal(sh.seed, ("trace",), P, sh.n_experts)).to(dev)
    x = torch.from_numpy(synth.activations_bf16(sh.seed, ("trace-x",), (P, sh.hidden)).view(np.int16)).to(dev).view(torch.bfloat16)
    ids, wts, prec = B.slicemoe_route_topk(logits, sh.top_k, rank_high=rank_high)
    y = torch.empty((P, sh.hidden), dtype=torch.float32, device=dev)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_launch = 400

    def layer(s):
        i, l = s % P, s % L
        B.slicemoe_layer(cs, tables[l], shared_tables[l], gate_vecs[l], x[i:i + 1], ids[i:i + 1], prec[i:i + 1], wts[i:i + 1],
                         ws, y=y[i:i + 1], flags=flags)

    for s in range(50):
        layer(s)
    e0.record()
    for s in range(n_launch):
        layer(s)
    e1.record()
    torch.cuda.synchronize()
    print(f"{name}: {e0.elapsed_time(e1) * 1e3 / n_launch:.2f} us per launch (plain stream launches, stamped kernel)")
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    n_cta = min(n_sm, 256)
    raw = np.zeros(n_cta * 256, dtype=np.int64)     # room for any number of stamps per CTA the library may have
    slots = ctypes.c_int(0)
    rc = B.lib().slicemoe_trace_read(raw.ctypes.data_as(c_void_p), n_cta, ctypes.byref(slots))
    if rc != 0:
        raise B.SliceMoEError(rc, "slicemoe_trace_read")
    out = raw[:n_cta * slots.value].reshape(n_cta, slots.value)
    props = torch.cuda.get_device_properties(0)
    clk = float(getattr(props, "clock_rate", 1965000)) / 1e3      # SM cycles per microsecond at the maximum clock
    dep = out[:, 1] / clk
    print("microseconds after the CTA's own dependency wait returned: mean / min / max over CTAs")
    order = [32, 33, 34, 35, 36, 37, 38, 39, 2, 3, 4, 5, 6, 7, 8, 12, 31, 18, 19, 40, 41, 42, 43, 44, 45, 46, 47, 9, 10, 14, 15, 16, 17, 23, 24, 25, 26, 11, 27, 28, 29, 30, 13]
    order += [k for k in range(48, out.shape[1])]   # stamps a working copy of the kernel may add
    for k in order:
        sel = out[:, k] != 0
        if sel.any():
            v = out[sel, k] / clk - dep[sel]
            print(f"  {NAMES.get(k, 'stamp %d' % k):36s} n {int(sel.sum()):3d}  {v.mean():6.2f} {v.min():6.2f} {v.max():6.2f}")
    if "--per-cta" in argv:   # one line per CTA: the gate/up phase's end per consumer group, last h value, y
        print("cta  gate/up done g0 g1 g2 g3 | last h | down tiles begin | digits g0..g3 | y written")
        for c in range(out.shape[0]):
            row = [out[c, k] / clk - dep[c] if out[c, k] > 0 else float("nan") for k in (5, 6, 7, 8, 12, 31, 14, 15, 16, 17, 13)]
            print(f"{c:3d}  " + " ".join(f"{v:6.2f}" for v in row))
    g = out[:, 20:23].astype(np.float64)
    t0 = g[:, 0].min()
    for label, col in (("kernel entry", 0), ("dependency wait over", 1), ("y written", 2)):
        v = g[:, col]
        v = (v[v > 0] - t0) / 1e3
        if v.size:
            print(f"  global timer, {label:22s} {v.min():7.2f} {v.mean():7.2f} {v.max():7.2f}")


if __name__ == "__main__":
    main(sys.argv[1:])
