"""Synthetic operator DAGs and clusters: the five benchmark shapes.

Each builder returns a :class:`Workload`: the problem data of the scheduling
model (operator set, precedence edges, durations, per-link-class communication
durations, memory adjustments, devices, link classes, capacities) plus the
recipe for drawing candidates.  Nothing here schedules anything; the arrays are
inputs for both the CUDA path and the CPU checker.
"""
from dataclasses import dataclass, field
from typing import Optional

import numpy as np

from . import rng

DEFAULT_SEED = 250309357

# stream ids of the counter-based generator (one per kind of draw)
_S_DUR, _S_COMM, _S_MEM, _S_DEG, _S_PRED, _S_NORM = 1, 2, 3, 4, 5, 6


@dataclass
class Workload:
    name: str
    num_ops: int                       # V = |I|
    num_devices: int                   # D = |J|
    edge_src: np.ndarray               # [E] int32, i1 of (i1, i2) in B
    edge_dst: np.ndarray               # [E] int32, i2
    dur: np.ndarray                    # [V] int32, D^o_i
    mem_delta: np.ndarray              # [V] int32, A_i
    comm: np.ndarray                   # [E, L] int32, D^c of edge e over link class l
    num_link_classes: int = 1          # L
    link_class: Optional[np.ndarray] = None   # [D, D] uint8 or None (all class 0)
    mem_weight: Optional[np.ndarray] = None   # [V] int32, W_i, or None (all 0)
    mem_capacity: Optional[np.ndarray] = None  # [D] int32 or None (no limit)
    num_candidates: int = 0            # K of the benchmark configuration
    assign_mode: str = "per_op"        # "per_op": x_c[i] uniform; "group_perm": x_c[i] = sigma_c(group[i])
    group: Optional[np.ndarray] = None  # [V] int32 group (pipeline slot) of each op, for "group_perm"
    meta: dict = field(default_factory=dict)

    @property
    def num_edges(self) -> int:
        return int(self.edge_src.shape[0])


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _node_link_classes(D: int, per_node: int) -> np.ndarray:
    node = np.arange(D) // per_node
    return np.ascontiguousarray((node[:, None] != node[None, :]).astype(np.uint8))


def tiny_pipeline(S: int = 4, M: int = 8, f: int = 2, b: int = 4, c: int = 1,
                  capacity: int = 8, K: int = 1024) -> Workload:
    """Config 1: S stages x M microbatches, ops F(s,m)=s*M+m, B(s,m)=S*M+s*M+m."""
    F = lambda s, m: s * M + m
    B = lambda s, m: S * M + s * M + m
    src, dst = [], []
    for m in range(M):
        for s in range(S - 1):
            src.append(F(s, m)); dst.append(F(s + 1, m))
    for m in range(M):
        src.append(F(S - 1, m)); dst.append(B(S - 1, m))
    for m in range(M):
        for s in range(S - 1):
            src.append(B(s + 1, m)); dst.append(B(s, m))
    V = 2 * S * M
    dur = np.concatenate([np.full(S * M, f), np.full(S * M, b)])
    A = np.concatenate([np.full(S * M, 1), np.full(S * M, -1)])
    E = len(src)
    return Workload(
        name="tiny_pipeline", num_ops=V, num_devices=S, edge_src=_i32(src), edge_dst=_i32(dst),
        dur=_i32(dur), mem_delta=_i32(A), comm=_i32(np.full((E, 1), c)),
        mem_capacity=_i32(np.full(S, capacity)), num_candidates=K,
        group=_i32(np.concatenate([np.repeat(np.arange(S), M)] * 2)),
        meta=dict(S=S, M=M, f=f, b=b, c=c))


def bidirectional_pipeline(P: int = 8, M: int = 20, K: int = 65536, seed: int = DEFAULT_SEED) -> Workload:
    """Config 2: P slots fed from both ends, M microbatches (first half travels
    0 -> P-1, second half P-1 -> 0), kinds F, B, W; op id = (kind*M + m)*P + p."""
    op = lambda kind, p, m: (kind * M + m) * P + p
    src, dst = [], []
    for m in range(M):
        path = list(range(P)) if m < M // 2 else list(range(P - 1, -1, -1))
        for a, b_ in zip(path[:-1], path[1:]):
            src.append(op(0, a, m)); dst.append(op(0, b_, m))
        src.append(op(0, path[-1], m)); dst.append(op(1, path[-1], m))
        back = path[::-1]
        for a, b_ in zip(back[:-1], back[1:]):
            src.append(op(1, a, m)); dst.append(op(1, b_, m))
        for p in range(P):
            src.append(op(1, p, m)); dst.append(op(2, p, m))
    V = 3 * M * P
    ids = np.arange(V)
    kind = ids // (M * P)
    dur = np.where(kind == 0, 10 + rng.randint(seed, _S_DUR, ids, 0, 0, 3),
                   np.where(kind == 1, 20 + rng.randint(seed, _S_DUR, ids, 0, 0, 3), 10))
    A = np.where(kind == 0, 2, -1)
    E = len(src)
    return Workload(
        name="bidirectional_pipeline", num_ops=V, num_devices=P, edge_src=_i32(src), edge_dst=_i32(dst),
        dur=_i32(dur), mem_delta=_i32(A), comm=_i32(np.full((E, 1), 2)),
        mem_capacity=_i32(np.full(P, 40)), num_candidates=K,
        assign_mode="group_perm", group=_i32(ids % P), meta=dict(P=P, M=M))


def bidirectional_unit(PP: int, M: int) -> Workload:
    """The bidirectional pipeline at the unit times of the paper's first experiment (Section V-A):
    T_f = T_i = T_w = 1 (forward, backward-for-input, backward-for-weights; a full backward is
    T_b = T_i + T_w = 2), stages = machines = PP, no communication time, and the memory limit
    "2 x parameters + (PP + 1) activations": every machine holds the parameters of its slot for both
    directions (W = 1 on one forward operator per slot and direction), an activation (A = +1) lives from a
    microbatch's forward operator to its weight-gradient operator (A = -1), capacity 2 + PP + 1.
    Same operator numbering and edges as `bidirectional_pipeline`; slot p belongs on machine p.
    The paper does not print its microbatch count, so M is the caller's choice."""
    w = bidirectional_pipeline(P=PP, M=M, K=1)
    V = w.num_ops
    ids = np.arange(V)
    kind, m_of = ids // (M * PP), (ids // PP) % M
    w.name = f"bidirectional_unit_PP{PP}_M{M}"
    w.dur = _i32(np.ones(V))
    w.comm = _i32(np.zeros_like(w.comm))
    w.mem_delta = _i32(np.where(kind == 0, 1, np.where(kind == 2, -1, 0)))
    w.mem_weight = _i32((kind == 0) & ((m_of == 0) | (m_of == M // 2)))
    w.mem_capacity = _i32(np.full(PP, 2 + PP + 1))
    return w


def _two_class_comm(seed, E):
    nbytes = rng.randint(seed, _S_COMM, np.arange(E), 0, 1, 64)
    return _i32(np.stack([(nbytes + 3) // 4, nbytes], axis=1))   # intra-node bw 4, inter-node bw 1


def _mirror_memory(seed, fwd_ops, bwd_of, V, lo, hi):
    A = np.zeros(V, dtype=np.int64)
    a = rng.randint(seed, _S_MEM, np.asarray(fwd_ops), 0, lo, hi)
    A[np.asarray(fwd_ops)] = a
    A[np.asarray(bwd_of)] = -a
    return A


def moe_branchy(layers: int = 32, experts: int = 8, microbatches: int = 4, K: int = 16384,
                seed: int = DEFAULT_SEED) -> Workload:
    """Config 3: per layer attention -> router -> `experts` parallel ops -> combine,
    forward then mirrored backward; D = 16 devices in 2 nodes of 8."""
    per_layer = experts + 3
    per_mb = 2 * layers * per_layer
    fwd = lambda mb, l, r: mb * per_mb + l * per_layer + r                     # r: 0 attn, 1 router, 2.. experts, last combine
    bwd = lambda mb, l, r: mb * per_mb + layers * per_layer + l * per_layer + r
    comb = per_layer - 1
    src, dst = [], []
    for mb in range(microbatches):
        for l in range(layers):
            src.append(fwd(mb, l, 0)); dst.append(fwd(mb, l, 1))
            for x in range(experts):
                src.append(fwd(mb, l, 1)); dst.append(fwd(mb, l, 2 + x))
                src.append(fwd(mb, l, 2 + x)); dst.append(fwd(mb, l, comb))
            if l + 1 < layers:
                src.append(fwd(mb, l, comb)); dst.append(fwd(mb, l + 1, 0))
        src.append(fwd(mb, layers - 1, comb)); dst.append(bwd(mb, layers - 1, comb))
        for l in range(layers - 1, -1, -1):
            for x in range(experts):
                src.append(bwd(mb, l, comb)); dst.append(bwd(mb, l, 2 + x))
                src.append(bwd(mb, l, 2 + x)); dst.append(bwd(mb, l, 1))
            src.append(bwd(mb, l, 1)); dst.append(bwd(mb, l, 0))
            if l > 0:
                src.append(bwd(mb, l, 0)); dst.append(bwd(mb, l - 1, comb))
    V = microbatches * per_mb
    ids = np.arange(V)
    u1 = rng.uniform01(seed, _S_NORM, ids, 0)
    u2 = rng.uniform01(seed, _S_NORM, ids, 1)
    normal = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)               # Box-Muller
    dur = np.maximum(1, np.rint(np.exp(3.0 + 0.5 * normal)).astype(np.int64))
    fwd_ops = [fwd(mb, l, r) for mb in range(microbatches) for l in range(layers) for r in range(per_layer)]
    bwd_ops = [bwd(mb, l, r) for mb in range(microbatches) for l in range(layers) for r in range(per_layer)]
    A = _mirror_memory(seed, fwd_ops, bwd_ops, V, 1, 4)
    D = 16
    return Workload(
        name="moe_branchy", num_ops=V, num_devices=D, edge_src=_i32(src), edge_dst=_i32(dst),
        dur=_i32(dur), mem_delta=_i32(A), comm=_two_class_comm(seed, len(src)), num_link_classes=2,
        link_class=_node_link_classes(D, 8), mem_capacity=_i32(np.full(D, 600)), num_candidates=K,
        meta=dict(layers=layers, experts=experts, microbatches=microbatches))


def multimodal_mimo(vision: int = 24, text: int = 32, decoder: int = 40, microbatches: int = 8,
                    K: int = 65536, seed: int = DEFAULT_SEED) -> Workload:
    """Config 4: vision and text encoder chains join at decoder layer 0; the backward
    pass mirrors it (decoder_b(0) feeds both encoder tails); D = 32 in 4 nodes of 8."""
    n_f = vision + text + decoder
    per_mb = 2 * n_f
    vf = lambda mb, l: mb * per_mb + l
    tf = lambda mb, l: mb * per_mb + vision + l
    df = lambda mb, l: mb * per_mb + vision + text + l
    vb = lambda mb, l: vf(mb, l) + n_f
    tb = lambda mb, l: tf(mb, l) + n_f
    db = lambda mb, l: df(mb, l) + n_f
    src, dst = [], []
    for mb in range(microbatches):
        for l in range(vision - 1):
            src.append(vf(mb, l)); dst.append(vf(mb, l + 1))
        for l in range(text - 1):
            src.append(tf(mb, l)); dst.append(tf(mb, l + 1))
        src.append(vf(mb, vision - 1)); dst.append(df(mb, 0))
        src.append(tf(mb, text - 1)); dst.append(df(mb, 0))
        for l in range(decoder - 1):
            src.append(df(mb, l)); dst.append(df(mb, l + 1))
        src.append(df(mb, decoder - 1)); dst.append(db(mb, decoder - 1))
        for l in range(decoder - 1, 0, -1):
            src.append(db(mb, l)); dst.append(db(mb, l - 1))
        src.append(db(mb, 0)); dst.append(vb(mb, vision - 1))
        src.append(db(mb, 0)); dst.append(tb(mb, text - 1))
        for l in range(vision - 1, 0, -1):
            src.append(vb(mb, l)); dst.append(vb(mb, l - 1))
        for l in range(text - 1, 0, -1):
            src.append(tb(mb, l)); dst.append(tb(mb, l - 1))
    V = microbatches * per_mb
    ids = np.arange(V)
    local = ids % n_f
    lo = np.where(local < vision, 6, np.where(local < vision + text, 4, 8))
    dur = lo + rng.randint(seed, _S_DUR, ids, 0, 0, 4)
    fwd_ops = [mb * per_mb + r for mb in range(microbatches) for r in range(n_f)]
    bwd_ops = [mb * per_mb + n_f + r for mb in range(microbatches) for r in range(n_f)]
    A = _mirror_memory(seed, fwd_ops, bwd_ops, V, 1, 3)
    D = 32
    return Workload(
        name="multimodal_mimo", num_ops=V, num_devices=D, edge_src=_i32(src), edge_dst=_i32(dst),
        dur=_i32(dur), mem_delta=_i32(A), comm=_two_class_comm(seed, len(src)), num_link_classes=2,
        link_class=_node_link_classes(D, 8), mem_capacity=_i32(np.full(D, 120)), num_candidates=K,
        meta=dict(vision=vision, text=text, decoder=decoder, microbatches=microbatches))


def random_layered(V: int = 16384, D: int = 64, K: Optional[int] = None, seed: int = DEFAULT_SEED) -> Workload:
    """Config 5: sqrt(V) layers of sqrt(V) ops (op id = layer*sqrt(V) + index); every op
    after layer 0 draws 1..3 distinct predecessors uniformly from all earlier layers."""
    side = int(round(V ** 0.5))
    if side * side != V:
        raise ValueError("V must be a perfect square")
    ids = np.arange(V)
    layer = ids // side
    earlier = layer * side                                     # number of ops in earlier layers
    deg = np.minimum(np.where(layer == 0, 0, rng.randint(seed, _S_DEG, ids, 0, 1, 3)), earlier)
    src, dst = [], []
    picks = []
    for t in range(3):
        # draw t-th predecessor among the `earlier - t` ids not yet taken (sequential sampling without replacement)
        n = np.maximum(earlier - t, 1)
        r = rng.rand64(seed, _S_PRED, ids, t) >> np.uint64(32)
        picks.append(((r * n.astype(np.uint64)) >> np.uint64(32)).astype(np.int64))
    p0 = picks[0]
    p1 = picks[1] + (picks[1] >= p0)
    lo2, hi2 = np.minimum(p0, p1), np.maximum(p0, p1)
    p2 = picks[2] + (picks[2] >= lo2)
    p2 = p2 + (p2 >= hi2)
    for t, p in enumerate((p0, p1, p2)):
        sel = deg > t
        src.append(p[sel]); dst.append(ids[sel])
    src = np.concatenate(src); dst = np.concatenate(dst)
    order = np.lexsort((src, dst))
    src, dst = src[order], dst[order]
    E = src.shape[0]
    if K is None:
        K = (1 << 30) // V
    return Workload(
        name=f"random_layered_V{V}_D{D}", num_ops=V, num_devices=D, edge_src=_i32(src), edge_dst=_i32(dst),
        dur=_i32(rng.randint(seed, _S_DUR, ids, 0, 1, 100)),
        mem_delta=_i32(rng.randint(seed, _S_MEM, ids, 0, -3, 3)),
        comm=_i32(rng.randint(seed, _S_COMM, np.arange(E), 0, 0, 20).reshape(E, 1)),
        mem_capacity=_i32(np.full(D, 1 << 20)), num_candidates=K, meta=dict(side=side))


SWEEP_POINTS = [(V, D) for V in (256, 1024, 4096, 16384) for D in (8, 64)]


def make_config(config: int, **kw) -> Workload:
    """The benchmark configurations by number (1..5); 5 takes V= and D=."""
    builders = {1: tiny_pipeline, 2: bidirectional_pipeline, 3: moe_branchy, 4: multimodal_mimo, 5: random_layered}
    return builders[config](**kw)
