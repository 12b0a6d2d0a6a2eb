"""Seeded synthetic workloads shaped like the paper's Flash / Pro serving profiles.

This module only *draws inputs*: request geometry (document lengths, request-order
permutation, protected token rows, which head of each output group is Global) from a
numpy PCG64 stream, and tensor values (latent KV stream, queries, projection weights,
a stand-in offline artifact) from one seeded torch generator.  It holds none of the
method's arithmetic, so both the CUDA path and the CPU checker can consume exactly the
same buffers without sharing any computation.

Geometry conventions (Section "Online position restoration and segmented merge"):
rows are kept in *packed* order -- document 0, 1, ..., D-1, then the query suffix --
which is the order of the packed latent stream.  Document i has length n_i and appears
in the request at offset delta_i; the query suffix is placed after all documents.
The protected set always contains every query-suffix row (the set Q of the
protected-row equation) plus a seeded fraction of document rows.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence

import numpy as np
import torch

GROUP_SIZE = 8       # logical heads per native output group (one of them is Global)
D_LATENT = 512       # kv_lora_rank: width of the shared latent c
D_ROPE = 64          # width of the rotary sub-vector
D_V = 128            # per-head value/output width after the up-projection W_uv


@dataclasses.dataclass
class Profile:
    n_heads: int
    n_groups: int
    o_rank: int                  # r_o: rows of each group's slice of W_a
    d_model: int                 # rows of W_b
    global_heads: np.ndarray     # [n_groups] absolute head index of each group's Global head
    sm_scale: float
    rope_base: float = 10000.0
    d_latent: int = D_LATENT
    d_rope: int = D_ROPE
    d_v: int = D_V
    group_size: int = GROUP_SIZE

    @property
    def n_local(self) -> int:
        return self.n_heads - self.n_groups

    @property
    def d_qk(self) -> int:
        return self.d_latent + self.d_rope

    @property
    def local_heads(self) -> np.ndarray:
        mask = np.ones(self.n_heads, dtype=bool)
        mask[self.global_heads] = False
        return np.nonzero(mask)[0].astype(np.int32)


@dataclasses.dataclass
class Layout:
    seg_off: np.ndarray           # int64 [S+1] packed-row prefix sums
    seg_delta: np.ndarray         # int64 [S]   request offset of each segment
    seg_has_artifact: np.ndarray  # uint8 [S]   0 for the query suffix

    @property
    def n_segs(self) -> int:
        return len(self.seg_delta)

    @property
    def n_rows(self) -> int:
        return int(self.seg_off[-1])

    @property
    def n_doc_rows(self) -> int:
        """Rows covered by the offline artifact tensor: up to the end of the last
        segment that has one."""
        has = np.nonzero(self.seg_has_artifact)[0]
        return int(self.seg_off[has[-1] + 1]) if len(has) else 0


@dataclasses.dataclass
class Workload:
    name: str
    seed: int
    profile: Profile
    layout: Layout
    prot_rows: np.ndarray                  # int32 [A] strictly ascending packed rows
    kv: torch.Tensor                       # bf16 [T, 576] = [c | k_rope at canonical position]
    q_g: torch.Tensor                      # bf16 [T, G, 576] queries of the Global heads
    q_l: torch.Tensor                      # bf16 [A, L, 576] queries of the Local heads on protected rows
    w_uv: torch.Tensor                     # bf16 [H, 128, 512]
    w_a: torch.Tensor                      # bf16 [G, r_o, 8*128]
    w_b: torch.Tensor                      # bf16 [d_model, G*r_o]
    z_off: torch.Tensor                    # bf16 [N_doc, G*r_o] stand-in offline artifact
    q_all: Optional[torch.Tensor] = None   # bf16 [T, H, 576] (small cases only)
    regime: str = "mandated"               # value regime the tensors were drawn in ("mandated" | "sharp")

    @property
    def T(self) -> int:
        return self.layout.n_rows

    @property
    def A(self) -> int:
        return len(self.prot_rows)


# ----------------------------------------------------------------------------------
# geometry
# ----------------------------------------------------------------------------------

def make_layout(doc_lens: Sequence[int], n_query: int, rng: Optional[np.random.Generator],
                shuffle: bool, base_delta: int = 0) -> Layout:
    """Documents in packed order 0..D-1; request order is a seeded permutation of them;
    delta_i is the prefix sum of lengths in request order.  Query suffix goes last."""
    doc_lens = [int(x) for x in doc_lens]
    D = len(doc_lens)
    order = np.arange(D)
    if shuffle and rng is not None and D > 1:
        order = rng.permutation(D)
    delta = np.zeros(D + 1, dtype=np.int64)
    run = int(base_delta)
    for d in order:
        delta[d] = run
        run += doc_lens[d]
    delta[D] = run
    seg_off = np.zeros(D + 2, dtype=np.int64)
    seg_off[1:D + 1] = np.cumsum(doc_lens)
    seg_off[D + 1] = seg_off[D] + int(n_query)
    has = np.ones(D + 1, dtype=np.uint8)
    has[D] = 0
    return Layout(seg_off=seg_off, seg_delta=delta, seg_has_artifact=has)


def draw_protected_rows(layout: Layout, pct_bp: int, rng: np.random.Generator,
                        run_len: int = 1) -> np.ndarray:
    """Every row of a segment without artifact + floor(pct_bp * N_doc / 10000) document
    rows drawn without replacement (integer arithmetic).  With run_len > 1 the document
    rows come as whole run_len-aligned runs inside documents."""
    S = layout.n_segs
    doc_rows = []
    forced = []
    for i in range(S):
        r = np.arange(layout.seg_off[i], layout.seg_off[i + 1], dtype=np.int64)
        (doc_rows if layout.seg_has_artifact[i] else forced).append(r)
    doc_rows = np.concatenate(doc_rows) if doc_rows else np.zeros(0, np.int64)
    forced = np.concatenate(forced) if forced else np.zeros(0, np.int64)
    n_pick = (int(pct_bp) * len(doc_rows)) // 10000
    if run_len <= 1:
        picked = rng.choice(doc_rows, size=n_pick, replace=False) if n_pick else np.zeros(0, np.int64)
    else:
        n_runs = n_pick // run_len
        starts = []
        for i in range(S):
            if not layout.seg_has_artifact[i]:
                continue
            lo, hi = int(layout.seg_off[i]), int(layout.seg_off[i + 1])
            # run starts aligned to run_len relative to the document start, whole runs only
            starts.append(np.arange(lo, hi - run_len + 1, run_len, dtype=np.int64))
        starts = np.concatenate(starts)
        chosen = rng.choice(starts, size=n_runs, replace=False) if n_runs else np.zeros(0, np.int64)
        picked = (chosen[:, None] + np.arange(run_len, dtype=np.int64)[None, :]).reshape(-1)
    rows = np.unique(np.concatenate([picked, forced]))
    return rows.astype(np.int32)


def draw_global_heads(n_groups: int, rng: np.random.Generator) -> np.ndarray:
    """The paper fixes one Global head per group of eight but not which; a random slot per
    group exercises every slice of W_a."""
    return (GROUP_SIZE * np.arange(n_groups) + rng.integers(0, GROUP_SIZE, size=n_groups)).astype(np.int32)


# ----------------------------------------------------------------------------------
# named configurations (the five benchmark shapes)
# ----------------------------------------------------------------------------------

CONFIGS = {
    # name: heads, groups, documents, query, protected basis points, run length, r_o, d_model, seed
    "tiny":      dict(H=16,  G=2,  docs=[256, 256],  shuffle=False, n_q=64,   pct_bp=500, run_len=1,  r_o=256,  d_model=1024, seed=0),
    "flash1":    dict(H=64,  G=8,  docs=[4096] * 8,  shuffle=True,  n_q=1024, pct_bp=300, run_len=1,  r_o=1024, d_model=4096, seed=1),
    "flash32k":  dict(H=64,  G=8,  docs="u16",       shuffle=True,  n_q=2048, pct_bp=None, run_len=1, r_o=1024, d_model=4096, seed=2),
    "flash256k": dict(H=64,  G=8,  docs=[4096] * 64, shuffle=True,  n_q=2048, pct_bp=200, run_len=16, r_o=1024, d_model=4096, seed=3),
    "pro128k":   dict(H=128, G=16, docs=[4096] * 32, shuffle=True,  n_q=4096, pct_bp=300, run_len=1,  r_o=1024, d_model=7168, seed=4),
    # not one of the five benchmark shapes: the longest context the paper's length table names (440K), with ragged
    # document lengths, as a parity case for long requests
    "flash440k": dict(H=64,  G=8,  docs=[4096] * 100 + [3000, 4500, 5000, 2999, 7777, 4100], shuffle=True, n_q=2048,
                      pct_bp=200, run_len=16, r_o=1024, d_model=4096, seed=5),
}
N_LAYERS_FLASH32K = 37


def make_geometry(name: str, layer: int = 0, seed: Optional[int] = None, pct_bp: Optional[int] = None):
    """Returns (profile, layout, prot_rows) for a named configuration.  For 'flash32k'
    every layer shares the layout (one request) but draws its own protected rows with a
    fraction uniform in [2 %, 5 %].  pct_bp overrides the configuration's protected share
    (basis points of the document rows), e.g. the controller budgets 1000 / 2000 / 2500."""
    cfg = CONFIGS[name]
    seed = cfg["seed"] if seed is None else seed
    rng = np.random.default_rng(np.random.PCG64(seed))
    docs = cfg["docs"]
    if isinstance(docs, str):  # 16 documents, integer lengths uniform in [1024, 4096]
        docs = rng.integers(1024, 4097, size=16).tolist()
    layout = make_layout(docs, cfg["n_q"], rng, cfg["shuffle"])
    gh = draw_global_heads(cfg["G"], rng)
    override = pct_bp
    pct_bp = cfg["pct_bp"] if override is None else int(override)
    rng_rows = rng
    if pct_bp is None:
        rng_rows = np.random.default_rng(np.random.PCG64(seed * 1000 + layer))
        pct_bp = int(rng_rows.integers(200, 501))
    prot = draw_protected_rows(layout, pct_bp, rng_rows, cfg["run_len"])
    profile = Profile(n_heads=cfg["H"], n_groups=cfg["G"], o_rank=cfg["r_o"], d_model=cfg["d_model"],
                      global_heads=gh, sm_scale=float(1.0 / np.sqrt(D_V + D_ROPE)))
    return profile, layout, prot


# ----------------------------------------------------------------------------------
# tensor values
# ----------------------------------------------------------------------------------

def _normal(shape, std, gen, device):
    x = torch.empty(shape, dtype=torch.float32, device=device)
    x.normal_(0.0, 1.0, generator=gen)
    x.mul_(std)
    return x.to(torch.bfloat16)


def _normal_big(shape, std, gen, device, chunk_rows=1 << 16):
    """Same distribution as _normal, drawn in row chunks so the fp32 staging buffer stays
    small for multi-GB tensors."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    n = shape[0]
    for lo in range(0, n, chunk_rows):
        hi = min(n, lo + chunk_rows)
        out[lo:hi] = _normal((hi - lo,) + tuple(shape[1:]), std, gen, device)
    return out


def make_tensors(name: str, profile: Profile, layout: Layout, prot_rows: np.ndarray, seed: int,
                 device="cpu", regime: str = "mandated", with_q_all: bool = False,
                 z_off_std: float = 0.02, value_phase: bool = False) -> Workload:
    """regime 'mandated': bf16 N(0, 0.02) latents and weights, q ~ N(0, 1) (the stated
    benchmark values; softmax is then close to uniform).  regime 'sharp': latents N(0, 1),
    q ~ N(0, 1.2), so that logits have a standard deviation near 2 and any masking or
    relocation error changes the output at O(1).  value_phase: the output-phase variant, whose
    value is the whole stored row: W_uv is [H, 128, 576] (everything else is drawn as before, in
    the same order, so the other tensors of a seed do not depend on the flag up to W_uv)."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(int(seed) * 7919 + (0 if regime == "mandated" else 1))
    kv_std, q_std = (0.02, 1.0) if regime == "mandated" else (1.0, 1.2)
    T, A = layout.n_rows, len(prot_rows)
    H, G, L = profile.n_heads, profile.n_groups, profile.n_local
    dqk = profile.d_qk
    kv = _normal_big((T, dqk), kv_std, gen, dev)
    q_all = None
    if with_q_all:
        q_all = _normal_big((T, H, dqk), q_std, gen, dev)
        gh = torch.as_tensor(profile.global_heads.astype(np.int64), device=dev)
        lh = torch.as_tensor(profile.local_heads.astype(np.int64), device=dev)
        pr = torch.as_tensor(prot_rows.astype(np.int64), device=dev)
        q_g = q_all[:, gh, :].contiguous()
        q_l = q_all[pr][:, lh, :].contiguous()
    else:
        q_g = _normal_big((T, G, dqk), q_std, gen, dev)
        q_l = _normal_big((A, L, dqk), q_std, gen, dev)
    w_uv = _normal((H, profile.d_v, profile.d_qk if value_phase else profile.d_latent), 0.02, gen, dev)
    w_a = _normal((G, profile.o_rank, GROUP_SIZE * profile.d_v), 0.02, gen, dev)
    w_b = _normal((profile.d_model, G * profile.o_rank), 0.02, gen, dev)
    z_off = _normal_big((layout.n_doc_rows, G * profile.o_rank), z_off_std, gen, dev)
    return Workload(name=name, seed=seed, profile=profile, layout=layout, prot_rows=prot_rows,
                    kv=kv, q_g=q_g, q_l=q_l, w_uv=w_uv, w_a=w_a, w_b=w_b, z_off=z_off, q_all=q_all, regime=regime)


def make_workload(name: str, device="cpu", regime: str = "mandated", layer: int = 0,
                  with_q_all: bool = False, seed: Optional[int] = None, value_phase: bool = False) -> Workload:
    profile, layout, prot = make_geometry(name, layer=layer, seed=seed)
    base_seed = CONFIGS[name]["seed"] if seed is None else seed
    return make_tensors(name, profile, layout, prot, base_seed * 1000 + layer, device=device,
                        regime=regime, with_q_all=with_q_all, value_phase=value_phase)


def make_custom(doc_lens: Sequence[int], n_query: int, n_heads: int, n_groups: int, o_rank: int,
                d_model: int, pct_bp: int, seed: int, device="cpu", regime: str = "sharp",
                shuffle: bool = True, run_len: int = 1, with_q_all: bool = False,
                base_delta: int = 0, value_phase: bool = False) -> Workload:
    """Free-form small case for parity tests (ragged lengths, odd sizes)."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    layout = make_layout(doc_lens, n_query, rng, shuffle, base_delta=base_delta)
    gh = draw_global_heads(n_groups, rng)
    prot = draw_protected_rows(layout, pct_bp, rng, run_len)
    profile = Profile(n_heads=n_heads, n_groups=n_groups, o_rank=o_rank, d_model=d_model,
                      global_heads=gh, sm_scale=float(1.0 / np.sqrt(D_V + D_ROPE)))
    return make_tensors("custom", profile, layout, prot, seed, device=device, regime=regime,
                        with_q_all=with_q_all, value_phase=value_phase)


def sample_rows(layout: Layout, prot_rows: np.ndarray, n_random: int, seed: int,
                max_docs: int = 6) -> np.ndarray:
    """Deterministic row sample used for full-size parity and for timing the CPU checker:
    segment-edge rows (canonical index 0, 1, 127, 128, 129, n-2, n-1) of up to max_docs
    documents -- always the first and the last in request order -- the first, middle and
    last query-suffix rows, plus n_random seeded rows, half protected, half not."""
    rng = np.random.default_rng(np.random.PCG64(seed + 77))
    S = layout.n_segs
    docs = [i for i in range(S) if layout.seg_has_artifact[i]]
    picked: List[int] = []
    if docs:
        by_req = sorted(docs, key=lambda i: int(layout.seg_delta[i]))
        chosen = {by_req[0], by_req[-1]}
        rest = [d for d in by_req if d not in chosen]
        if rest and max_docs > 2:
            extra = rng.choice(rest, size=min(max_docs - 2, len(rest)), replace=False)
            chosen.update(int(e) for e in extra)
        for i in sorted(chosen):
            lo, n = int(layout.seg_off[i]), int(layout.seg_off[i + 1] - layout.seg_off[i])
            for c in (0, 1, 127, 128, 129, n - 2, n - 1):
                if 0 <= c < n:
                    picked.append(lo + c)
    for i in range(S):
        if not layout.seg_has_artifact[i]:
            lo, n = int(layout.seg_off[i]), int(layout.seg_off[i + 1] - layout.seg_off[i])
            picked += [lo, lo + n // 2, lo + n - 1]
    T = layout.n_rows
    is_prot = np.zeros(T, dtype=bool)
    is_prot[prot_rows] = True
    n_half = n_random // 2
    if n_half and len(prot_rows):
        picked += rng.choice(prot_rows, size=min(n_half, len(prot_rows)), replace=False).tolist()
    unprot = np.nonzero(~is_prot)[0]
    if n_random - n_half and len(unprot):
        picked += rng.choice(unprot, size=min(n_random - n_half, len(unprot)), replace=False).tolist()
    return np.unique(np.asarray(picked, dtype=np.int64))


# ----------------------------------------------------------------------------------
# inputs of the selection rules (Eq. protected, Eq. moe): seeded data only, no rule arithmetic
# ----------------------------------------------------------------------------------

def draw_policy_inputs(layout: Layout, seed: int, n_dirty: int = 64, tie_share: float = 0.05):
    """Dirty rows (any order, with a few duplicates) and float32 Indexer scores with exact ties:
    scores are standard normal, a `tie_share` of the rows is set to one of four fixed values."""
    rng = np.random.default_rng(seed)
    T = layout.n_rows
    dirty = rng.integers(0, T, size=n_dirty).astype(np.int32)
    if n_dirty >= 4:
        dirty[-2:] = dirty[:2]
    scores = rng.standard_normal(T).astype(np.float32)
    n_tie = int(tie_share * T)
    if n_tie:
        idx = rng.choice(T, size=n_tie, replace=False)
        scores[idx] = rng.choice(np.array([-0.5, 0.0, 0.25, 1.5], dtype=np.float32), size=n_tie)
    return dirty, scores


def draw_router_weights(n: int, seed: int, temperature: float = 1.5, tie_share: float = 0.02) -> np.ndarray:
    """Top-6 router weights [n, 6] float32 in arbitrary slot order: six shares of a softmax over
    random logits, scaled by the token's routed mass in (0.2, 0.9); a few rows carry exact ties."""
    rng = np.random.default_rng(seed)
    logits = rng.standard_normal((n, 6)) * temperature
    e = np.exp(logits - logits.max(axis=1, keepdims=True))
    p = e / e.sum(axis=1, keepdims=True) * rng.uniform(0.2, 0.9, size=(n, 1))
    p = p.astype(np.float32)
    n_tie = int(tie_share * n)
    if n_tie:
        rows = rng.choice(n, size=n_tie, replace=False)
        a, b = rng.integers(0, 6, size=n_tie), rng.integers(0, 6, size=n_tie)
        p[rows, a] = p[rows, b]
    return p


def make_random_request(seed: int, n_heads: int = 16, n_groups: int = 2, o_rank: int = 256, d_model: int = 512,
                        regime: str = "sharp", device="cpu", value_phase: bool = False) -> Workload:
    """A seeded irregular request for edge-case parity: 2-7 segments whose lengths mix tile-boundary
    values (1, 2, 63..65, 127..129, 255..257) with random ones, a random request order with random gaps
    between segments, some segments in the middle without artifact (new rows), a short query suffix
    last in the request, and a random share of protected document rows."""
    rng = np.random.default_rng(np.random.PCG64(1000 + seed))
    special = [1, 2, 63, 64, 65, 127, 128, 129, 255, 256, 257]
    n_docs = int(rng.integers(2, 7))
    lens = [int(rng.choice(special)) if rng.random() < 0.6 else int(rng.integers(3, 600)) for _ in range(n_docs)]
    lens.append(int(rng.integers(1, 80)))                    # query suffix, packed last
    has = np.ones(n_docs + 1, dtype=np.uint8)
    has[n_docs] = 0
    for i in range(n_docs):
        if rng.random() < 0.2:
            has[i] = 0                                       # a new (uncached) segment in the middle
    if has[:n_docs].sum() == 0:
        has[0] = 1
    order = list(rng.permutation(n_docs)) + [n_docs]         # request order; the query comes last
    delta = np.zeros(n_docs + 1, dtype=np.int64)
    run = int(rng.integers(0, 3)) * int(rng.integers(0, 40))
    for i in order:
        delta[i] = run
        run += lens[i] + (int(rng.integers(0, 50)) if rng.random() < 0.4 else 0)
    seg_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    layout = Layout(seg_off=seg_off, seg_delta=delta, seg_has_artifact=has)
    prot = draw_protected_rows(layout, int(rng.integers(0, 3000)), rng)
    profile = Profile(n_heads=n_heads, n_groups=n_groups, o_rank=o_rank, d_model=d_model,
                      global_heads=draw_global_heads(n_groups, rng), sm_scale=float(1.0 / np.sqrt(D_V + D_ROPE)))
    return make_tensors("random", profile, layout, prot, seed, device=device, regime=regime, value_phase=value_phase)
