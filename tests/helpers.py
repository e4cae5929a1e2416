"""Shared by the GPU parity tests: builds the same seeded layer for the oracle (numpy) and for the
CUDA path (packed on the GPU by slicemoe_pack), and the error metrics of the tolerance."""
from __future__ import annotations

import numpy as np

from paper_2512_12990_b200 import synth

REL_L2_TOL = 1e-3          # ||y - y_ref||_2 / ||y_ref||_2
MAX_ABS_TOL = 2e-3         # max |y - y_ref| / rms(y_ref)


def errors(y: np.ndarray, y_ref: np.ndarray):
    y = np.asarray(y, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    rel_l2 = np.linalg.norm(y - y_ref) / max(np.linalg.norm(y_ref), 1e-300)
    rms = np.sqrt(np.mean(y_ref ** 2))
    max_abs = np.abs(y - y_ref).max() / max(rms, 1e-300)
    return rel_l2, max_abs


def assert_close(y, y_ref, what=""):
    rel_l2, max_abs = errors(y, y_ref)
    assert rel_l2 <= REL_L2_TOL and max_abs <= MAX_ABS_TOL, f"{what}: rel_l2={rel_l2:.3e} max_abs/rms={max_abs:.3e}"
    return rel_l2, max_abs


class Layer:
    """One seeded MoE layer, held twice: oracle dicts (CPU) and packed device buffers (GPU).

    Only the experts in `needed` (plus two decoys) are generated; every other slot of the device expert
    table points at a decoy, so that a wrong expert id shows up as a numerical mismatch."""

    def __init__(self, shape: synth.Shape, needed, layer: int = 0, device="cuda", b_high: int = 8, b_low: int = 4):
        import torch
        from oracle import amat
        from paper_2512_12990_b200 import binding as B
        self.shape = shape
        self.cshape = B.make_shape(shape.hidden, shape.inter, shape.n_experts, shape.top_k, shape.group,
                                   shape.n_shared, shape.shared_inter, shape.shared_sigmoid_gate, b_high, b_low)
        needed = sorted(set(int(e) for e in needed))
        decoys = [e for e in range(shape.n_experts) if e not in needed][:1]
        self.oracle_experts = {}
        self.packed = {}
        self._keep = []

        def make(tag, inter):
            W = synth.expert_weights(shape.seed, layer, tag, shape.hidden, inter)
            o = {k: amat.pack_matrix(W[k], shape.group, b_high, b_low) for k in ("gate", "up", "down")}
            d = {}
            for k in ("gate", "up", "down"):
                Wd = torch.from_numpy(W[k]).to(device)
                d[k] = B.slicemoe_pack(Wd, shape.group, b_high, b_low)
            return o, d

        for e in needed + decoys:
            self.oracle_experts[e], self.packed[e] = make(e, shape.inter)
        fill = self.packed[decoys[0]] if decoys else self.packed[needed[0]]
        table = [self.packed.get(e, fill) for e in range(shape.n_experts)]
        self.experts_tbl = B.expert_table(table, device)
        self.oracle_shared, self.packed_shared = [], []
        for j in range(shape.n_shared):
            o, d = make(f"shared{j}", shape.shared_inter)
            self.oracle_shared.append(o)
            self.packed_shared.append(d)
        self.shared_tbl = B.expert_table(self.packed_shared, device) if shape.n_shared else None
        self.gate_vec = None
        self.gate_vec_dev = None
        if shape.shared_sigmoid_gate:
            self.gate_vec = synth.normal_f32(shape.seed, ("gate_vec", layer), (shape.hidden,), 0.02)
            self.gate_vec_dev = torch.from_numpy(self.gate_vec).to(device)
        self.ws = B.new_workspace(self.cshape, device)

    def oracle_list(self):
        """Indexable by expert id (only generated experts are present)."""
        return self.oracle_experts


def x_inputs(shape: synth.Shape, T: int, tag="x"):
    """bf16 activations: (uint16 bits [T, hidden], float64 values)."""
    bits = synth.activations_bf16(shape.seed, (tag,), (T, shape.hidden))
    return bits, synth.bf16_to_f64(bits)


def to_dev_bf16(bits: np.ndarray, device="cuda"):
    import torch
    return torch.from_numpy(bits.view(np.int16).copy()).to(device).view(torch.bfloat16)


def oracle_mat_from_device(pm) -> dict:
    """The oracle's view (canonical arrays, as oracle.amat.pack_matrix returns them) of a matrix packed on the
    GPU, read back through slicemoe_unpack_plane / slicemoe_unpack_meta.  For the large configurations, where
    packing every matrix a second time in numpy would take minutes; slicemoe_pack itself is compared bit for bit
    with the oracle's quantiser in test_gpu_pack.py."""
    from paper_2512_12990_b200 import binding as B
    msb = B.slicemoe_unpack_plane(pm.msb, pm.N, pm.K).cpu().numpy()
    lsb = B.slicemoe_unpack_plane(pm.lsb, pm.N, pm.K).cpu().numpy()
    s, z = B.slicemoe_unpack_meta(pm.scale, pm.zp, pm.N, pm.K, pm.group)
    return dict(scale=s.cpu().numpy(), zp=z.cpu().numpy(), msb=msb, lsb=lsb, group=pm.group, b_high=8, b_low=4)


def oracle_expert_from_device(packed: dict) -> dict:
    return {k: oracle_mat_from_device(packed[k]) for k in ("gate", "up", "down")}


def device_expert(seed: int, tag, hidden: int, inter: int, group: int, std: float = 0.02) -> dict:
    """One SwiGLU expert drawn on the GPU (torch generator seeded by (seed, tag)) and packed there."""
    import hashlib
    import torch
    from paper_2512_12990_b200 import binding as B
    gen = torch.Generator(device="cuda")
    gen.manual_seed(int.from_bytes(hashlib.sha256(repr((seed, tag)).encode()).digest()[:7], "little"))
    out = {}
    for name, shape in (("gate", (inter, hidden)), ("up", (inter, hidden)), ("down", (hidden, inter))):
        out[name] = B.slicemoe_pack(torch.randn(shape, device="cuda", generator=gen) * std, group)
    return out
