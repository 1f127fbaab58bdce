"""Synthetic training-state layouts: which rank holds which box of which tensor.

The rules restate how the paper describes LFM training states (Appendix A and Sec. 3.2):
GEMM weights are split along the output or the input dimension by tensor parallelism while
norms are replicated; pipeline parallelism only decides which rank holds a layer; the
distributed optimizer flattens and concatenates a rank's (TP-local) tensors and splits the
flat buffer evenly over the data-parallel group, so that slices start and end in the middle
of rows; replicated shards are saved once, by the holder with the smallest load so far
(Sec. 4.1, worst-fit balancing).  The output is metadata only: nothing here touches tensor
bytes or knows how a reshard is executed.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

from .meta import BOX, DTYPE_BF16, DTYPE_F32, FLAT_SLICE, ShardMeta, ShardedState, prod

ALIGN = 256  # every saved shard starts on a 256-byte boundary of its rank buffer


def align_up(x: int, a: int = ALIGN) -> int:
    return (x + a - 1) // a * a


# --------------------------------------------------------------------------- model specs
@dataclass
class TensorSpec:
    fqn: str
    shape: Tuple[int, ...]
    tp: str = "rep"  # "rep" | "col" (split dim 0) | "row" (split dim 1)
    parts: Optional[Tuple[int, ...]] = None  # fused tensors: dim-0 sizes split one by one
    layer: int = -1  # -1: before the first layer (stage 0); -2: after the last (last stage)
    expert: int = -1  # expert index for expert parallelism, -1 = not an expert tensor
    unit: int = 0  # FSDP flat unit this tensor is concatenated into


@dataclass
class ModelSpec:
    name: str
    tensors: List[TensorSpec]
    n_layers: int
    n_experts: int = 0

    @property
    def n_params(self) -> int:
        return sum(prod(t.shape) for t in self.tensors)


def gpt_model(name: str, L: int, H: int, F: int, V: int, P: int) -> ModelSpec:
    """GPT with learned positions, LayerNorm with bias, fused QKV, tied embedding."""
    ts: List[TensorSpec] = [
        TensorSpec("embedding.word.weight", (V, H), "col"),
        TensorSpec("embedding.position.weight", (P, H), "rep"),
    ]
    for i in range(L):
        p = f"layers.{i}."
        ts += [
            TensorSpec(p + "ln1.weight", (H,), "rep", layer=i),
            TensorSpec(p + "ln1.bias", (H,), "rep", layer=i),
            TensorSpec(p + "attn.qkv.weight", (3 * H, H), "col", (H, H, H), layer=i),
            TensorSpec(p + "attn.qkv.bias", (3 * H,), "col", (H, H, H), layer=i),
            TensorSpec(p + "attn.proj.weight", (H, H), "row", layer=i),
            TensorSpec(p + "attn.proj.bias", (H,), "rep", layer=i),
            TensorSpec(p + "ln2.weight", (H,), "rep", layer=i),
            TensorSpec(p + "ln2.bias", (H,), "rep", layer=i),
            TensorSpec(p + "mlp.fc1.weight", (F, H), "col", layer=i),
            TensorSpec(p + "mlp.fc1.bias", (F,), "col", layer=i),
            TensorSpec(p + "mlp.fc2.weight", (H, F), "row", layer=i),
            TensorSpec(p + "mlp.fc2.bias", (H,), "rep", layer=i),
        ]
    ts += [
        TensorSpec("final_ln.weight", (H,), "rep", layer=-2),
        TensorSpec("final_ln.bias", (H,), "rep", layer=-2),
    ]
    return ModelSpec(name, ts, L)


def llama_model(name: str, L: int, H: int, nq: int, nkv: int, F: int, V: int, *, fused: bool,
                tied: bool, fsdp_units: bool = False) -> ModelSpec:
    """Llama-style decoder: RMSNorm, GQA, SwiGLU.  `fused` packs QKV and gate/up (dim 0)."""
    hd = H // nq
    q, kv = nq * hd, nkv * hd
    root = L  # FSDP: layers are units 0..L-1, the root unit (embedding + final norm) is unit L
    ts: List[TensorSpec] = [TensorSpec("embed_tokens.weight", (V, H), "col", unit=root)]
    for i in range(L):
        p = f"layers.{i}."
        u = i if fsdp_units else 0
        ts.append(TensorSpec(p + "input_norm.weight", (H,), "rep", layer=i, unit=u))
        if fused:
            ts.append(TensorSpec(p + "attn.qkv.weight", (q + 2 * kv, H), "col", (q, kv, kv), layer=i, unit=u))
        else:
            ts += [
                TensorSpec(p + "attn.q.weight", (q, H), "col", layer=i, unit=u),
                TensorSpec(p + "attn.k.weight", (kv, H), "col", layer=i, unit=u),
                TensorSpec(p + "attn.v.weight", (kv, H), "col", layer=i, unit=u),
            ]
        ts.append(TensorSpec(p + "attn.o.weight", (H, q), "row", layer=i, unit=u))
        ts.append(TensorSpec(p + "post_norm.weight", (H,), "rep", layer=i, unit=u))
        if fused:
            ts.append(TensorSpec(p + "mlp.gate_up.weight", (2 * F, H), "col", (F, F), layer=i, unit=u))
        else:
            ts += [
                TensorSpec(p + "mlp.gate.weight", (F, H), "col", layer=i, unit=u),
                TensorSpec(p + "mlp.up.weight", (F, H), "col", layer=i, unit=u),
            ]
        ts.append(TensorSpec(p + "mlp.down.weight", (H, F), "row", layer=i, unit=u))
    ts.append(TensorSpec("final_norm.weight", (H,), "rep", layer=-2, unit=root))
    if not tied:
        ts.append(TensorSpec("lm_head.weight", (V, H), "col", layer=-2, unit=root))
    return ModelSpec(name, ts, L)


def moe_model(name: str, L: int, H: int, E: int, F: int, V: int) -> ModelSpec:
    """Decoder with unfused attention and E SwiGLU experts per layer, untied head."""
    ts: List[TensorSpec] = [TensorSpec("embed_tokens.weight", (V, H), "rep")]
    for i in range(L):
        p = f"layers.{i}."
        ts.append(TensorSpec(p + "input_norm.weight", (H,), "rep", layer=i))
        for n in ("q", "k", "v", "o"):
            ts.append(TensorSpec(p + f"attn.{n}.weight", (H, H), "rep", layer=i))
        ts.append(TensorSpec(p + "post_norm.weight", (H,), "rep", layer=i))
        ts.append(TensorSpec(p + "router.weight", (E, H), "rep", layer=i))
        for e in range(E):
            q = p + f"experts.{e}."
            ts += [
                TensorSpec(q + "gate.weight", (F, H), "rep", layer=i, expert=e),
                TensorSpec(q + "up.weight", (F, H), "rep", layer=i, expert=e),
                TensorSpec(q + "down.weight", (H, F), "rep", layer=i, expert=e),
            ]
    ts.append(TensorSpec("final_norm.weight", (H,), "rep", layer=-2))
    ts.append(TensorSpec("lm_head.weight", (V, H), "rep", layer=-2))
    return ModelSpec(name, ts, L, n_experts=E)


# --------------------------------------------------------------------------- parallelism
@dataclass
class Parallelism:
    tp: int = 1
    pp: int = 1
    dp: int = 1
    ep: int = 1  # expert parallelism; expert ranks take the place of data-parallel ranks
    zero: str = "none"  # "none": optimizer states whole, replicated over dp
    #                      "zero1": one flat buffer per model-parallel rank, split over dp
    #                      "fsdp": one flat buffer per unit, split over dp; no params entry
    #                              unless `fsdp_params` (then params are flat-split too)

    @property
    def world(self) -> int:
        return self.tp * self.pp * self.dp * self.ep

    def rank(self, tp: int, pp: int, dp: int, ep: int = 0) -> int:
        # tp fastest, then ep, then dp, then pp (Megatron-style order)
        return ((pp * self.dp + dp) * self.ep + ep) * self.tp + tp

    def __str__(self) -> str:
        s = f"TP{self.tp}.PP{self.pp}.DP{self.dp}"
        if self.ep > 1:
            s += f".EP{self.ep}"
        if self.zero != "none":
            s += f".{self.zero}"
        return s


Box = Tuple[Tuple[int, ...], Tuple[int, ...]]  # (offsets, lengths) in global coordinates


def _split(n: int, parts: int, i: int) -> Tuple[int, int]:
    """[begin, end) of chunk i when n is cut into `parts` nearly equal chunks."""
    return n * i // parts, n * (i + 1) // parts


def local_pieces(t: TensorSpec, tp: int, r: int) -> List[Box]:
    """Boxes of the global tensor whose concatenation (C order, dim 0) is TP rank r's local tensor."""
    shape = t.shape
    nd = len(shape)
    if t.tp == "rep" or tp == 1:
        return [((0,) * nd, tuple(shape))]
    if t.tp == "col":
        parts = t.parts if t.parts else (shape[0],)
        out, base = [], 0
        for s in parts:
            b, e = _split(s, tp, r)
            if e > b:
                out.append(((base + b,) + (0,) * (nd - 1), (e - b,) + tuple(shape[1:])))
            base += s
        return out
    if t.tp == "row":
        b, e = _split(shape[1], tp, r)
        if e <= b:
            return []
        return [((0, b) + (0,) * (nd - 2), (shape[0], e - b) + tuple(shape[2:]))]
    raise ValueError(t.tp)


def stage_of(t: TensorSpec, n_layers: int, pp: int) -> int:
    if t.layer == -1:
        return 0
    if t.layer == -2:
        return pp - 1
    return t.layer * pp // n_layers


# --------------------------------------------------------------------------- state dicts
@dataclass
class StateKinds:
    param_dtype: Optional[Tuple[int, int]] = (2, DTYPE_BF16)  # (itemsize, tag) or None: no params
    optim: Tuple[str, ...] = ("master", "exp_avg", "exp_avg_sq")  # fp32 states per param
    optim_dtype: Tuple[int, int] = (4, DTYPE_F32)


@dataclass
class _Shard:
    """One saved shard before placement: entries that sit back to back in a rank buffer."""

    key: tuple  # identity for de-duplication
    holders: List[int]
    entries: List[ShardMeta]  # buf_index / byte_offset filled at placement

    @property
    def nbytes(self) -> int:
        return sum(e.byte_length for e in self.entries)


def _collect_shards(model: ModelSpec, par: Parallelism, kinds: StateKinds) -> List[_Shard]:
    """Every shard any rank holds, in registration order, with the ranks that hold it."""
    shards: Dict[tuple, _Shard] = {}
    order: List[tuple] = []

    def add(key: tuple, rank: int, make_entries) -> None:
        s = shards.get(key)
        if s is None:
            s = _Shard(key, [], make_entries())
            shards[key] = s
            order.append(key)
        s.holders.append(rank)

    for pp in range(par.pp):
        for dp in range(par.dp):
            for ep in range(par.ep):
                for tp in range(par.tp):
                    rank = par.rank(tp, pp, dp, ep)
                    mine: List[Tuple[TensorSpec, List[Box]]] = []
                    for t in model.tensors:
                        if stage_of(t, model.n_layers, par.pp) != pp:
                            continue
                        if t.expert >= 0 and par.ep > 1:
                            if t.expert * par.ep // model.n_experts != ep:
                                continue
                        pieces = local_pieces(t, par.tp, tp)
                        if pieces:
                            mine.append((t, pieces))
                    # model parameters: whole local tensors, replicated over dp
                    if kinds.param_dtype is not None and par.zero != "fsdp":
                        isz, tag = kinds.param_dtype
                        for t, pieces in mine:
                            key = ("p", t.fqn, tuple(pieces))
                            add(key, rank, lambda t=t, pieces=pieces: [
                                ShardMeta(t.fqn, isz, tag, tuple(t.shape), o, l) for (o, l) in pieces])
                    # optimizer states
                    isz, tag = kinds.optim_dtype
                    if par.zero == "none":
                        for kind in kinds.optim:
                            for t, pieces in mine:
                                fqn = f"optim.{kind}.{t.fqn}"
                                key = ("o", fqn, tuple(pieces))
                                add(key, rank, lambda t=t, pieces=pieces, fqn=fqn: [
                                    ShardMeta(fqn, isz, tag, tuple(t.shape), o, l) for (o, l) in pieces])
                    else:
                        units = sorted({t.unit for t, _ in mine}) if par.zero == "fsdp" else [None]
                        for kind in kinds.optim:
                            for u in units:
                                group = [(t, p) for (t, p) in mine if u is None or t.unit == u]
                                total = sum(prod(l) for _, ps in group for (_, l) in ps)
                                slice_len = -(-total // par.dp)  # ceil: the tail rank may own less
                                lo, hi = dp * slice_len, min((dp + 1) * slice_len, total)
                                pos = 0
                                for t, pieces in group:
                                    fqn = f"optim.{kind}.{t.fqn}"
                                    for (o, l) in pieces:
                                        n = prod(l)
                                        a, b = max(lo, pos), min(hi, pos + n)
                                        if b > a:
                                            fb, fe = a - pos, b - pos
                                            key = ("z", fqn, o, l, fb, fe, kind, u, a - lo)
                                            add(key, rank, lambda t=t, fqn=fqn, o=o, l=l, fb=fb, fe=fe: [
                                                ShardMeta(fqn, isz, tag, tuple(t.shape), o, l,
                                                          kind=FLAT_SLICE, flat_begin=fb, flat_end=fe)])
                                        pos += n
    return [shards[k] for k in order]


def _region_id(s: _Shard) -> tuple:
    """Entries with the same region id on one rank are stored back to back (one flat slice)."""
    if s.key[0] == "z":
        return ("z", s.key[6], s.key[7])  # (state kind, unit)
    return s.key


def build_state(model: ModelSpec, par: Parallelism, kinds: StateKinds, *, dedup: bool) -> ShardedState:
    """Metadata of the training state under `par`.

    dedup=True  : the saved side; a shard held by several ranks is stored once, by the holder
                  with the smallest cumulative bytes so far (worst fit, registration order).
    dedup=False : the wanted side; every rank materialises everything it holds.
    Rank buffers are laid out in registration order; a region (a local tensor, or a rank's
    flat slice of one state kind and unit) starts on a 256-byte boundary and its entries are
    consecutive.
    """
    shards = _collect_shards(model, par, kinds)
    world = par.world
    per_rank: List[List[_Shard]] = [[] for _ in range(world)]
    load = [0] * world
    for s in shards:
        if dedup:
            owner = min(s.holders, key=lambda r: (load[r], r))
            load[owner] += s.nbytes
            per_rank[owner].append(s)
        else:
            for r in s.holders:
                per_rank[r].append(s)
    state = ShardedState()
    for r in range(world):
        off = 0
        last_region = None
        for s in per_rank[r]:
            reg = _region_id(s)
            if reg != last_region:
                off = align_up(off)
                last_region = reg
            for e in s.entries:
                m = ShardMeta(e.fqn, e.itemsize, e.dtype_tag, e.global_shape, e.offsets, e.lengths,
                              r, off, e.kind, e.flat_begin, e.flat_end)
                state.metas.append(m)
                off += m.byte_length
        state.buf_bytes.append(align_up(off))
    return state


@dataclass
class ReshardCase:
    """A saved state, a wanted state, and how to fill the saved bytes."""

    name: str
    src: ShardedState
    dst: ShardedState
    fill: str = "index"  # "index" | "uniform" | "normal"
    seed: int = 0
    note: str = ""
    # (kind, saved dtype tag, wanted dtype tag) when tensors change their element type on the
    # way (kind 1: binary32 -> bfloat16, kind 2: the reverse); None: bytes are moved unchanged
    convert: Optional[Tuple[int, int, int]] = None

    @property
    def plan_opts(self) -> Dict[str, int]:
        """Planner options this case needs (none unless it converts)."""
        if self.convert is None:
            return {}
        return dict(convert=self.convert[0], convert_src_tag=self.convert[1], convert_dst_tag=self.convert[2])

    @property
    def key_ids(self) -> Dict[str, int]:
        names = sorted({m.fqn for m in self.src.metas} | {m.fqn for m in self.dst.metas})
        return {n: i for i, n in enumerate(names)}


def reshard_case(name: str, model: ModelSpec, src_par: Parallelism, dst_par: Parallelism,
                 kinds: StateKinds, fill: str = "index", seed: int = 0, note: str = "") -> ReshardCase:
    return ReshardCase(name, build_state(model, src_par, kinds, dedup=True),
                       build_state(model, dst_par, kinds, dedup=False), fill, seed, note)
