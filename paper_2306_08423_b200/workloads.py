"""Seeded synthetic inputs: event tables and search spaces.

This module only *draws inputs*.  It holds none of the simulator's arithmetic
(no timeline, no schedule, no cost formula) and is the one module that both the
CUDA engine's callers and the CPU oracle's tests may import; it imports neither
of them.

An event table stands in for the output of DistSim's event generator and event
profiler (paper Sec. 4.1-4.2): for every event class (mp, b) - model-parallel
degree and micro-batch size, i.e. the operator's parameters and input shape that
key an event - it gives each layer's forward and backward computation time in
integer nanoseconds, plus the alpha-beta constants that replace profiled
communication events.  The workloads below stand in for the paper's BERT-Large /
GPT-2 / T5 / BERT-exLarge / 145B-GPT profiles (Sec. 5-6), which are not
available; shapes, sizes and value distributions follow the five benchmark
configurations.

Random numbers come from SplitMix64 (Steele, Lea, Flood 2014; public-domain
reference by Vigna): state += 0x9E3779B97F4A7C15, then two xor-shift-multiply
rounds.  Integers uniform in [lo, hi] are ``lo + x mod (hi - lo + 1)``.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

_MASK = (1 << 64) - 1

M_RULE_DIVIDES, M_RULE_CEIL = 0, 1
PARTITION_BALANCED, PARTITION_ALL = 0, 1
SCHED_GPIPE, SCHED_1F1B = 0, 1


class SplitMix64:
    def __init__(self, seed: int):
        self.state = seed & _MASK

    def next(self) -> int:
        self.state = (self.state + 0x9E3779B97F4A7C15) & _MASK
        z = self.state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
        return z ^ (z >> 31)

    def randint(self, lo: int, hi: int) -> int:
        return lo + self.next() % (hi - lo + 1)

    def normal(self) -> float:
        """Box-Muller from two draws; u1 in (0, 1], u2 in [0, 1)."""
        u1 = ((self.next() >> 11) + 1) / float(1 << 53)
        u2 = (self.next() >> 11) / float(1 << 53)
        return math.sqrt(-2.0 * math.log(u1)) * math.cos(2.0 * math.pi * u2)


@dataclass
class SearchSpace:
    mp_max: int
    pp_max: int
    m_list: np.ndarray                      # int32, ascending
    m_rule: int = M_RULE_DIVIDES
    partition_mode: int = PARTITION_BALANCED
    sched_mask: int = 3                     # bit 0 GPipe, bit 1 1F1B, bit 2 asynchronous 1F1B,
                                            # bit 3 interleaved 1F1B with v = 2, 4, .. v_max chunks per device
    v_max: int = 0

    def __post_init__(self):
        self.m_list = np.ascontiguousarray(self.m_list, dtype=np.int32)


@dataclass
class EventTable:
    n_layers: int
    n_devices: int
    gpus_per_node: int
    global_batch: int
    seq: int
    hidden: int
    class_mp: np.ndarray                    # int32 [n_classes]
    class_b: np.ndarray                     # int32 [n_classes]
    fwd_ns: np.ndarray                      # int64 [n_classes, n_layers]
    bwd_ns: np.ndarray                      # int64 [n_classes, n_layers]
    layer_is_expert: np.ndarray             # uint8 [n_layers]
    grad_bytes: np.ndarray                  # int64 [n_layers], at mp = 1
    alpha_intra_ns: int = 2_000
    beta_intra: int = 300                   # bytes per ns (300 GB/s)
    alpha_inter_ns: int = 10_000
    beta_inter: int = 25                    # bytes per ns (25 GB/s)
    dp_bucket_bytes: int = 25 * 2**20
    dp_overlap: int = 1
    act_bytes_per_elem: int = 2             # bf16 messages
    allreduce_profile_max: int = 0          # k > 0: all-reduces over more than k devices are the
                                            # k-device time scaled by the volume formula (paper Sec. 4.2)
    jitter_fwd_ns: np.ndarray = None        # int64 [P, stages] or None: extra time of the forward
    jitter_bwd_ns: np.ndarray = None        # (backward) item of micro-batch j on stage d is [j mod P, d]

    def __post_init__(self):
        self.class_mp = np.ascontiguousarray(self.class_mp, dtype=np.int32)
        self.class_b = np.ascontiguousarray(self.class_b, dtype=np.int32)
        self.fwd_ns = np.ascontiguousarray(self.fwd_ns, dtype=np.int64)
        self.bwd_ns = np.ascontiguousarray(self.bwd_ns, dtype=np.int64)
        self.layer_is_expert = np.ascontiguousarray(self.layer_is_expert, dtype=np.uint8)
        self.grad_bytes = np.ascontiguousarray(self.grad_bytes, dtype=np.int64)
        if self.jitter_fwd_ns is not None:
            self.jitter_fwd_ns = np.ascontiguousarray(self.jitter_fwd_ns, dtype=np.int64)
            self.jitter_bwd_ns = np.ascontiguousarray(self.jitter_bwd_ns, dtype=np.int64)
            assert self.jitter_fwd_ns.ndim == 2 and self.jitter_fwd_ns.shape == self.jitter_bwd_ns.shape
        assert self.fwd_ns.shape == (self.n_classes, self.n_layers)
        assert self.bwd_ns.shape == (self.n_classes, self.n_layers)

    @property
    def n_classes(self) -> int:
        return int(self.class_mp.shape[0])


@dataclass
class Workload:
    name: str
    table: EventTable
    space: SearchSpace
    seed: int
    top_k: int = 0                          # > 0: how many fastest candidates to emit
    notes: dict = field(default_factory=dict)


def _pow2_upto(n: int):
    v = 1
    while v <= n:
        yield v
        v *= 2


def event_classes(n_devices: int, global_batch: int, n_layers: int, space: SearchSpace):
    """Every (mp, micro-batch size) shape a strategy of the space can present to
    the profiler, sorted: the set of distinct events that must be timed."""
    classes = set()
    for mp in _pow2_upto(space.mp_max):
        for pp in _pow2_upto(min(space.pp_max, n_layers)):
            if n_devices % (mp * pp):
                continue
            dp = n_devices // (mp * pp)
            if global_batch % dp:
                continue
            bp = global_batch // dp
            for m in space.m_list.tolist():
                if m < 1 or m > bp:
                    continue
                if space.m_rule == M_RULE_DIVIDES and bp % m:
                    continue
                classes.add((mp, -(-bp // m)))
    return sorted(classes)


def space_shape(table, space):
    """Rows of the search space for reporting: a list of (mp, pp, dp, [valid m], partitions,
    schedules, v) in canonical order; v = 1 for the plain schedules, the number of model chunks
    per device for a row of interleaved candidates (which has one schedule and partitions the
    layers into pp * v virtual stages); a row of bidirectional-pipeline candidates (sched_mask
    bit 4: one schedule, even m, v = 1) follows the interleaved rows of its (mp, pp).  Pure counting; candidates = sum(len(ms) * partitions *
    schedules)."""
    rows = []
    n_sched = bin(space.sched_mask & 7).count("1")
    v_max = int(getattr(space, "v_max", 0)) if space.sched_mask & 8 else 0
    for mp in _pow2_upto(space.mp_max):
        for pp in _pow2_upto(min(space.pp_max, table.n_layers)):
            if table.n_devices % (mp * pp):
                continue
            dp = table.n_devices // (mp * pp)
            if table.global_batch % dp:
                continue
            bp = table.global_batch // dp
            ms = [m for m in space.m_list.tolist()
                  if 1 <= m <= bp and (space.m_rule == M_RULE_CEIL or bp % m == 0)]
            if ms and n_sched:
                parts = 1 if space.partition_mode == PARTITION_BALANCED else math.comb(table.n_layers - 1, pp - 1)
                rows.append((mp, pp, dp, ms, parts, n_sched, 1))
            if pp < 2:
                continue
            for v in _pow2_upto(v_max):
                if v < 2 or pp * v > min(64, table.n_layers):
                    continue
                mv = [m for m in ms if m % pp == 0]
                if not mv:
                    continue
                parts = 1 if space.partition_mode == PARTITION_BALANCED else math.comb(table.n_layers - 1, pp * v - 1)
                rows.append((mp, pp, dp, mv, parts, 1, v))
            if space.sched_mask & 16:
                # bidirectional pipelines: half of the micro-batches each way, pp stages
                me = [m for m in ms if m % 2 == 0]
                if me:
                    parts = 1 if space.partition_mode == PARTITION_BALANCED else math.comb(table.n_layers - 1, pp - 1)
                    rows.append((mp, pp, dp, me, parts, 1, 1))
    return rows


def count_candidates_and_cells(table, space):
    """(candidates, recurrence cells) of a space; a candidate has 2 * m * pp * v cells (one per
    schedule item: forward and backward of every micro-batch on every (virtual) stage)."""
    cands = cells = 0
    for mp, pp, dp, ms, parts, n_sched, v in space_shape(table, space):
        cands += len(ms) * parts * n_sched
        cells += sum(2 * m * pp * v for m in ms) * parts * n_sched
    return cands, cells


def build_table(*, per_sample_fwd_ns, per_sample_bwd_extra_ns, n_devices, gpus_per_node,
                global_batch, seq, hidden, space, layer_is_expert=None, grad_bytes=None,
                **cluster) -> EventTable:
    """Expands per-sample, mp=1 layer times into the per-class table.

    The drawn time is per sample at mp = 1; an event of class (mp, b) takes
    ``b * ceil(t / mp)`` forward and ``b * ceil((2 t + u) / mp)`` backward.  The
    engines only ever see the expanded table, so measured (non-linear) profiles
    would load unchanged."""
    f1 = [int(v) for v in per_sample_fwd_ns]
    u = [int(v) for v in per_sample_bwd_extra_ns]
    n_layers = len(f1)
    classes = event_classes(n_devices, global_batch, n_layers, space)
    fwd = np.zeros((len(classes), n_layers), dtype=np.int64)
    bwd = np.zeros((len(classes), n_layers), dtype=np.int64)
    for k, (mp, b) in enumerate(classes):
        for l in range(n_layers):
            fwd[k, l] = b * (-(-f1[l] // mp))
            bwd[k, l] = b * (-(-(2 * f1[l] + u[l]) // mp))
    if layer_is_expert is None:
        layer_is_expert = np.zeros(n_layers, dtype=np.uint8)
    if grad_bytes is None:
        grad_bytes = np.full(n_layers, 12 * hidden * hidden * 2, dtype=np.int64)
    return EventTable(
        n_layers=n_layers, n_devices=n_devices, gpus_per_node=gpus_per_node,
        global_batch=global_batch, seq=seq, hidden=hidden,
        class_mp=np.array([c[0] for c in classes], dtype=np.int32),
        class_b=np.array([c[1] for c in classes], dtype=np.int32),
        fwd_ns=fwd, bwd_ns=bwd, layer_is_expert=layer_is_expert, grad_bytes=grad_bytes,
        **cluster)


def _uniform_layers(rng: SplitMix64, n_layers: int, lo: int, hi: int):
    f1 = [rng.randint(lo, hi) for _ in range(n_layers)]
    u = [rng.randint(0, 20_000) for _ in range(n_layers)]
    return f1, u


def config0(seed: int = 0) -> Workload:
    """Tiny search: 8 devices (2 nodes x 4), 12 layers, h=768, s=512, B=32."""
    space = SearchSpace(mp_max=8, pp_max=4, m_list=[1, 2, 4, 8, 16, 32],
                        m_rule=M_RULE_DIVIDES, partition_mode=PARTITION_BALANCED)
    f1, u = _uniform_layers(SplitMix64(seed), 12, 200_000, 400_000)
    table = build_table(per_sample_fwd_ns=f1, per_sample_bwd_extra_ns=u, n_devices=8,
                        gpus_per_node=4, global_batch=32, seq=512, hidden=768, space=space)
    return Workload("config0_tiny", table, space, seed)


def config1(seed: int = 1) -> Workload:
    """64 devices (8 x 8), 24 layers, h=1024, s=1024, B=512; every composition."""
    space = SearchSpace(mp_max=8, pp_max=16, m_list=[1, 2, 4, 8, 16, 32, 64, 128],
                        m_rule=M_RULE_DIVIDES, partition_mode=PARTITION_ALL)
    f1, u = _uniform_layers(SplitMix64(seed), 24, 200_000, 400_000)
    table = build_table(per_sample_fwd_ns=f1, per_sample_bwd_extra_ns=u, n_devices=64,
                        gpus_per_node=8, global_batch=512, seq=1024, hidden=1024, space=space)
    return Workload("config1_64dev_all_compositions", table, space, seed)


def config2(seed: int = 2) -> Workload:
    """1024 devices (128 x 8), 96 layers, h=12288, s=2048, B=1536; long pipelines."""
    space = SearchSpace(mp_max=8, pp_max=64, m_list=np.arange(1, 257),
                        m_rule=M_RULE_CEIL, partition_mode=PARTITION_BALANCED)
    f1, u = _uniform_layers(SplitMix64(seed), 96, 8_000_000, 12_000_000)
    table = build_table(per_sample_fwd_ns=f1, per_sample_bwd_extra_ns=u, n_devices=1024,
                        gpus_per_node=8, global_batch=1536, seq=2048, hidden=12288, space=space)
    return Workload("config2_1024dev_gpt3like", table, space, seed)


def config3(seed: int = 3) -> Workload:
    """256 devices (32 x 8), 48-layer MoE-like model, lognormal layer times."""
    space = SearchSpace(mp_max=8, pp_max=4, m_list=[4, 8, 16, 32, 64],
                        m_rule=M_RULE_DIVIDES, partition_mode=PARTITION_ALL)
    rng = SplitMix64(seed)
    n_layers = 48
    expert = np.array([l % 2 for l in range(n_layers)], dtype=np.uint8)
    f1 = []
    for l in range(n_layers):
        median = 900_000.0 if expert[l] else 300_000.0
        f1.append(max(1, int(round(median * math.exp(0.5 * rng.normal())))))
    u = [rng.randint(0, 20_000) for _ in range(n_layers)]
    table = build_table(per_sample_fwd_ns=f1, per_sample_bwd_extra_ns=u, n_devices=256,
                        gpus_per_node=8, global_batch=4096, seq=1024, hidden=2048, space=space,
                        layer_is_expert=expert)
    return Workload("config3_256dev_moe", table, space, seed)


def config4(seed: int = 2) -> Workload:
    """Timeline emission: the 1024 fastest candidates of config 2."""
    w = config2(seed)
    return Workload("config4_emit_top1024_of_config2", w.table, w.space, seed, top_k=1024)


def paper_grid(seed: int = 7) -> Workload:
    """The shape of the paper's own strategy search (Sec. 6): 16 GPUs on 4 nodes, a 48-layer
    transformer, global batch 16, every degree in {1, 2, 4, 8, 16}, with all-reduces above 8
    devices extrapolated from the 8-device time (Sec. 4.2).  Event times are synthetic."""
    space = SearchSpace(mp_max=16, pp_max=16, m_list=[1, 2, 4, 8, 16], m_rule=M_RULE_DIVIDES,
                        partition_mode=PARTITION_BALANCED)
    f1, u = _uniform_layers(SplitMix64(seed), 48, 200_000, 400_000)
    table = build_table(per_sample_fwd_ns=f1, per_sample_bwd_extra_ns=u, n_devices=16,
                        gpus_per_node=4, global_batch=16, seq=512, hidden=1024, space=space,
                        allreduce_profile_max=8)
    return Workload("paper_grid_16gpu_48layers", table, space, seed)


def add_jitter(w: Workload, slots: int, max_ns: int, seed: int = 11) -> Workload:
    """Gives a workload a per-micro-batch jitter table: `slots` (a power of two) micro-batch
    slots x pp_max stages of extra item time, uniform in [0, max_ns]."""
    rng = SplitMix64(seed)
    stages = w.space.pp_max
    w.table.jitter_fwd_ns = np.array([[rng.randint(0, max_ns) for _ in range(stages)] for _ in range(slots)], np.int64)
    w.table.jitter_bwd_ns = np.array([[rng.randint(0, max_ns) for _ in range(stages)] for _ in range(slots)], np.int64)
    w.name += f"_jitter{slots}"
    return w


CONFIGS = {0: config0, 1: config1, 2: config2, 3: config3, 4: config4}


def random_small(seed: int, *, n_devices=8, gpus_per_node=4, n_layers=6, global_batch=16,
                 seq=64, hidden=32, mp_max=4, pp_max=4, m_list=(1, 2, 3, 4, 8),
                 m_rule=M_RULE_CEIL, partition_mode=PARTITION_ALL, moe=True,
                 dp_bucket_bytes=3000, dp_overlap=1, lo=50, hi=5000, sched_mask=3, v_max=0) -> Workload:
    """Small irregular workload for element-by-element parity tests."""
    rng = SplitMix64(seed)
    space = SearchSpace(mp_max=mp_max, pp_max=pp_max, m_list=list(m_list), m_rule=m_rule,
                        partition_mode=partition_mode, sched_mask=sched_mask, v_max=v_max)
    f1 = [rng.randint(lo, hi) for _ in range(n_layers)]
    u = [rng.randint(0, hi // 4) for _ in range(n_layers)]
    expert = np.array([(rng.next() & 1) if moe else 0 for _ in range(n_layers)], dtype=np.uint8)
    grad = np.array([rng.randint(1, 4 * dp_bucket_bytes if dp_bucket_bytes else 10_000)
                     for _ in range(n_layers)], dtype=np.int64)
    table = build_table(per_sample_fwd_ns=f1, per_sample_bwd_extra_ns=u, n_devices=n_devices,
                        gpus_per_node=gpus_per_node, global_batch=global_batch, seq=seq,
                        hidden=hidden, space=space, layer_is_expert=expert, grad_bytes=grad,
                        dp_bucket_bytes=dp_bucket_bytes, dp_overlap=dp_overlap,
                        alpha_intra_ns=rng.randint(0, 50), beta_intra=rng.randint(1, 64),
                        alpha_inter_ns=rng.randint(50, 500), beta_inter=rng.randint(1, 8))
    return Workload(f"random_small_{seed}", table, space, seed)
