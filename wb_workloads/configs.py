"""The five benchmark configurations (plus parity-only variants) as concrete layouts.

Each layout is stated twice, independently:
  * as a slice list (the source map handed to the library and to the oracle), built
    from explicit rectangle arithmetic on `Param` row blocks;
  * as a procedural ``load_weights`` written with torch tensor ops.
The id probe of Section 3.1 (fill the checkpoint with global ids, load, compare)
checks one against the other in the tests.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Iterator, List, Tuple

import torch
import torch.nn.functional as F

from .rng import SplitMix64
from .types import (WB_BF16, WB_F32, CkptTensor, Layout, LoaderGroup, Workload)

CONFIG_NAMES = ["cfg1", "cfg1b", "cfg1c", "cfg2", "cfg3", "cfg4", "cfg5"]


# --------------------------------------------------------------------------------------
# model shapes
# --------------------------------------------------------------------------------------
@dataclass
class ModelSpec:
    L: int
    H: int
    nq: int
    nkv: int
    hd: int
    F: int
    V: int
    E: int = 0     # experts per layer (0 = dense)
    Fe: int = 0    # expert FFN width


def build_ckpt(spec: ModelSpec) -> Tuple[List[CkptTensor], Dict[str, int]]:
    """Checkpoint tensor table in canonical order; every tensor is a row-major [out, in]
    matrix, vectors are [1, n]."""
    ck: List[CkptTensor] = []
    idx: Dict[str, int] = {}

    def add(name, r, c):
        idx[name] = len(ck)
        ck.append(CkptTensor(name, r, c))

    s = spec
    add("embed_tokens", s.V, s.H)
    for l in range(s.L):
        p = f"layers.{l}."
        add(p + "q_proj", s.nq * s.hd, s.H)
        add(p + "k_proj", s.nkv * s.hd, s.H)
        add(p + "v_proj", s.nkv * s.hd, s.H)
        add(p + "o_proj", s.H, s.nq * s.hd)
        if s.E:
            add(p + "router", s.E, s.H)
            for e in range(s.E):
                add(p + f"experts.{e}.gate_proj", s.Fe, s.H)
                add(p + f"experts.{e}.up_proj", s.Fe, s.H)
                add(p + f"experts.{e}.down_proj", s.H, s.Fe)
        else:
            add(p + "gate_proj", s.F, s.H)
            add(p + "up_proj", s.F, s.H)
            add(p + "down_proj", s.H, s.F)
        add(p + "input_norm", 1, s.H)
        add(p + "post_attn_norm", 1, s.H)
    add("final_norm", 1, s.H)
    add("lm_head", s.V, s.H)
    return ck, idx


# --------------------------------------------------------------------------------------
# slice-list side: parameters as stacks of checkpoint row blocks
# --------------------------------------------------------------------------------------
@dataclass
class Param:
    """A local row-major [rows, cols] parameter assembled from row blocks; block =
    (local_row0, nrows, ckpt_index, ckpt_r0, ckpt_c0) and spans the full local width."""
    rows: int
    cols: int
    blocks: List[Tuple[int, int, int, int, int]]

    @property
    def numel(self) -> int:
        return self.rows * self.cols


def roundup(x: int, m: int) -> int:
    return (x + m - 1) // m * m


def flat_range_rects(cols: int, b: int, e: int) -> List[Tuple[int, int, int, int, int]]:
    """Row-major flat range [b, e) of a matrix with `cols` columns as <= 3 rectangles
    (r0, c0, nr, nc, flat_start)."""
    if e <= b:
        return []
    rb, cb = divmod(b, cols)
    re_, ce = divmod(e, cols)
    if rb == re_:
        return [(rb, cb, 1, e - b, b)]
    out = []
    if cb:
        out.append((rb, cb, 1, cols - cb, b))
        rb += 1
    if re_ > rb:
        out.append((rb, 0, re_ - rb, cols, rb * cols))
    if ce:
        out.append((re_, 0, 1, ce, re_ * cols))
    return out


class _SliceWriter:
    def __init__(self, layout: Layout, ckpt: List[CkptTensor]):
        self.layout = layout
        self.ckpt = ckpt

    def dense(self, name: str, rank: int, dtype: int, p: Param) -> None:
        """Local tensor `name` holds exactly parameter p."""
        t = self.layout.add_tensor(name, rank, dtype, p.numel)
        for (row0, nrows, ck, cr0, cc0) in p.blocks:
            c = self.ckpt[ck]
            self.layout.add_slice(t, row0 * p.cols, p.cols, 1, ck, c.rows, c.cols,
                                  cr0, cc0, nrows, p.cols)

    def flat_unit(self, names: List[str], ranks: List[int], dtype: int,
                  params: List[Param]) -> None:
        """FlatParameter-style unit: params flattened and concatenated in order to length
        N, cut into W = len(names) shards of length roundup(ceil(N/W), 128); shard k holds
        flat [kL, min((k+1)L, N)) followed by padding."""
        W = len(names)
        N = sum(p.numel for p in params)
        L = roundup(-(-N // W), 128)
        tens = [self.layout.add_tensor(names[k], ranks[k], dtype, L) for k in range(W)]
        P0 = 0
        for p in params:
            for k in range(W):
                b = max(k * L, P0)
                e = min((k + 1) * L, N, P0 + p.numel)
                for (lr0, lc0, lnr, lnc, fstart) in flat_range_rects(p.cols, b - P0, e - P0):
                    for (row0, nrows, ck, cr0, cc0) in p.blocks:
                        a = max(lr0, row0)
                        z = min(lr0 + lnr, row0 + nrows)
                        if z <= a:
                            continue
                        c = self.ckpt[ck]
                        self.layout.add_slice(
                            tens[k], P0 + a * p.cols + lc0 - k * L, p.cols, 1,
                            ck, c.rows, c.cols, cr0 + (a - row0), cc0 + lc0, z - a, lnc)
            P0 += p.numel


def _fsdp_shards(flat: torch.Tensor, W: int) -> List[torch.Tensor]:
    """Procedural twin of `_SliceWriter.flat_unit`: pad and view as [W, L]."""
    N = flat.numel()
    L = roundup(-(-N // W), 128)
    pad = -1 if not flat.dtype.is_floating_point else 0
    padded = F.pad(flat, (0, W * L - N), value=pad)
    return list(padded.view(W, L).unbind(0))


# ---- Megatron-style trainer parameters (rank t of T) -------------------------------------
def _mega_qkv(s: ModelSpec, ix, l, t, T) -> Param:
    Q = s.nq // s.nkv
    Gt = s.nkv // T
    p = f"layers.{l}."
    blocks = []
    for j in range(Gt):
        g = t * Gt + j
        b = j * (Q + 2) * s.hd
        blocks.append((b, Q * s.hd, ix[p + "q_proj"], g * Q * s.hd, 0))
        blocks.append((b + Q * s.hd, s.hd, ix[p + "k_proj"], g * s.hd, 0))
        blocks.append((b + (Q + 1) * s.hd, s.hd, ix[p + "v_proj"], g * s.hd, 0))
    return Param((Q + 2) * s.hd * Gt, s.H, blocks)


def _rowblock(ix, name, rows, cols, t, T) -> Param:
    return Param(rows // T, cols, [(0, rows // T, ix[name], t * (rows // T), 0)])


def _colblock(ix, name, rows, cols, t, T) -> Param:
    return Param(rows, cols // T, [(0, rows, ix[name], 0, t * (cols // T))])


def _whole(ix, name, rows, cols) -> Param:
    return Param(rows, cols, [(0, rows, ix[name], 0, 0)])


def _mega_layer_params(s: ModelSpec, ix, l, t, T, fused=True) -> List[Tuple[str, Param]]:
    p = f"layers.{l}."
    out: List[Tuple[str, Param]] = []
    if fused:
        out.append(("linear_qkv", _mega_qkv(s, ix, l, t, T)))
    else:
        out.append(("q", _rowblock(ix, p + "q_proj", s.nq * s.hd, s.H, t, T)))
        out.append(("k", _rowblock(ix, p + "k_proj", s.nkv * s.hd, s.H, t, T)))
        out.append(("v", _rowblock(ix, p + "v_proj", s.nkv * s.hd, s.H, t, T)))
    out.append(("linear_proj", _colblock(ix, p + "o_proj", s.H, s.nq * s.hd, t, T)))
    if fused:
        Ft = s.F // T
        out.append(("linear_fc1", Param(2 * Ft, s.H, [
            (0, Ft, ix[p + "gate_proj"], t * Ft, 0),
            (Ft, Ft, ix[p + "up_proj"], t * Ft, 0)])))
    else:
        out.append(("gate", _rowblock(ix, p + "gate_proj", s.F, s.H, t, T)))
        out.append(("up", _rowblock(ix, p + "up_proj", s.F, s.H, t, T)))
    out.append(("linear_fc2", _colblock(ix, p + "down_proj", s.H, s.F, t, T)))
    out.append(("input_norm", _whole(ix, p + "input_norm", 1, s.H)))
    out.append(("post_attn_norm", _whole(ix, p + "post_attn_norm", 1, s.H)))
    return out


def _mega_layer_tensors(s: ModelSpec, ts: List[torch.Tensor], t, T, fused=True):
    """Procedural twin of `_mega_layer_params` (tensor ops only)."""
    q, k, v, o, gate, up, down, n1, n2 = ts
    Q = s.nq // s.nkv
    out = []
    if fused:
        qg = q.view(s.nkv, Q * s.hd, s.H)
        kg = k.view(s.nkv, s.hd, s.H)
        vg = v.view(s.nkv, s.hd, s.H)
        grouped = torch.cat([qg, kg, vg], dim=1)            # [nkv, (Q+2)hd, H]
        out.append(("linear_qkv", grouped.chunk(T, dim=0)[t].reshape(-1, s.H)))
    else:
        out += [("q", q.chunk(T, 0)[t]), ("k", k.chunk(T, 0)[t]), ("v", v.chunk(T, 0)[t])]
    out.append(("linear_proj", o.chunk(T, dim=1)[t]))
    if fused:
        out.append(("linear_fc1", torch.cat([gate.chunk(T, 0)[t], up.chunk(T, 0)[t]], 0)))
    else:
        out += [("gate", gate.chunk(T, 0)[t]), ("up", up.chunk(T, 0)[t])]
    out.append(("linear_fc2", down.chunk(T, dim=1)[t]))
    out.append(("input_norm", n1))
    out.append(("post_attn_norm", n2))
    return out


_DENSE_LAYER = ["q_proj", "k_proj", "v_proj", "o_proj", "gate_proj", "up_proj", "down_proj",
                "input_norm", "post_attn_norm"]


# --------------------------------------------------------------------------------------
# trainer layouts
# --------------------------------------------------------------------------------------
def trainer_tp_fsdp(s: ModelSpec, ck, ix, T: int, W: int, dtype: int, fused=True):
    """Megatron TP=T, each TP rank's parameters in FSDP=W flat shards; rank = tp*W + dp."""
    lay = Layout("trainer")
    w = _SliceWriter(lay, ck)
    for t in range(T):
        ranks = [t * W + d for d in range(W)]
        w.flat_unit([f"t{r}.embed.flat" for r in ranks], ranks, dtype,
                    [_rowblock(ix, "embed_tokens", s.V, s.H, t, T)])
        for l in range(s.L):
            w.flat_unit([f"t{r}.layers.{l}.flat" for r in ranks], ranks, dtype,
                        [p for _, p in _mega_layer_params(s, ix, l, t, T, fused)])
        w.flat_unit([f"t{r}.final.flat" for r in ranks], ranks, dtype,
                    [_whole(ix, "final_norm", 1, s.H), _rowblock(ix, "lm_head", s.V, s.H, t, T)])
    lay.freeze()

    def groups() -> Iterator[LoaderGroup]:
        def embed(ts):
            out = {}
            for t in range(T):
                sh = _fsdp_shards(ts[0].chunk(T, 0)[t].reshape(-1), W)
                for d in range(W):
                    out[f"t{t * W + d}.embed.flat"] = sh[d]
            return out
        yield [ix["embed_tokens"]], embed
        for l in range(s.L):
            def layer(ts, l=l):
                out = {}
                for t in range(T):
                    flat = torch.cat([p.reshape(-1) for _, p in _mega_layer_tensors(s, ts, t, T, fused)])
                    sh = _fsdp_shards(flat, W)
                    for d in range(W):
                        out[f"t{t * W + d}.layers.{l}.flat"] = sh[d]
                return out
            yield [ix[f"layers.{l}.{n}"] for n in _DENSE_LAYER], layer

        def final(ts):
            out = {}
            for t in range(T):
                flat = torch.cat([ts[0].reshape(-1), ts[1].chunk(T, 0)[t].reshape(-1)])
                sh = _fsdp_shards(flat, W)
                for d in range(W):
                    out[f"t{t * W + d}.final.flat"] = sh[d]
            return out
        yield [ix["final_norm"], ix["lm_head"]], final
    return lay, groups


def _nonexpert_layer_names(s: ModelSpec) -> List[str]:
    if s.E:
        return ["q_proj", "k_proj", "v_proj", "o_proj", "router", "input_norm", "post_attn_norm"]
    return _DENSE_LAYER


def trainer_fsdp(s: ModelSpec, ck, ix, W: int, dtype: int, EP: int = 0):
    """Pure FSDP=W over unsplit checkpoint tensors in checkpoint order; with EP > 0 the
    experts are kept out of the flat units and held as per-rank stacks instead."""
    lay = Layout("trainer")
    w = _SliceWriter(lay, ck)
    ranks = list(range(W))

    def whole(name):
        c = ck[ix[name]]
        return _whole(ix, name, c.rows, c.cols)

    w.flat_unit([f"t{r}.embed.flat" for r in ranks], ranks, dtype, [whole("embed_tokens")])
    for l in range(s.L):
        p = f"layers.{l}."
        w.flat_unit([f"t{r}.layers.{l}.flat" for r in ranks], ranks, dtype,
                    [whole(p + n) for n in _nonexpert_layer_names(s)])
        if s.E:
            per = s.E // EP
            for k in range(EP):
                for kind, rows, cols in (("gate", s.Fe, s.H), ("up", s.Fe, s.H), ("down", s.H, s.Fe)):
                    blocks = [(i * rows, rows, ix[p + f"experts.{k * per + i}.{kind}_proj"], 0, 0)
                              for i in range(per)]
                    w.dense(f"t{k}.layers.{l}.{kind}_local", k, dtype, Param(per * rows, cols, blocks))
    w.flat_unit([f"t{r}.final.flat" for r in ranks], ranks, dtype, [whole("final_norm"), whole("lm_head")])
    lay.freeze()

    def groups() -> Iterator[LoaderGroup]:
        def unit(tag):
            def fn(ts):
                sh = _fsdp_shards(torch.cat([t.reshape(-1) for t in ts]), W)
                return {f"t{r}.{tag}.flat": sh[r] for r in ranks}
            return fn
        yield [ix["embed_tokens"]], unit("embed")
        for l in range(s.L):
            p = f"layers.{l}."
            yield [ix[p + n] for n in _nonexpert_layer_names(s)], unit(f"layers.{l}")
            if s.E:
                per = s.E // EP
                for kind in ("gate", "up", "down"):
                    def experts(ts, l=l, kind=kind):
                        stacked = torch.stack(ts, 0)                  # [E, rows, cols]
                        return {f"t{k}.layers.{l}.{kind}_local": c
                                for k, c in enumerate(stacked.chunk(EP, 0))}
                    yield [ix[p + f"experts.{e}.{kind}_proj"] for e in range(s.E)], experts
        yield [ix["final_norm"], ix["lm_head"]], unit("final")
    return lay, groups


def trainer_tp_pp(s: ModelSpec, ck, ix, T: int, P: int, dtype: int):
    """Megatron TP=T x PP=P, every parameter its own dense local tensor; rank = pp*T + tp.
    Stage 0 also holds the embedding, the last stage final_norm and the output layer."""
    lay = Layout("trainer")
    w = _SliceWriter(lay, ck)
    per_stage = s.L // P
    for t in range(T):
        w.dense(f"t{t}.word_embeddings", t, dtype, _rowblock(ix, "embed_tokens", s.V, s.H, t, T))
    for l in range(s.L):
        pp = l // per_stage
        for t in range(T):
            r = pp * T + t
            for nm, p in _mega_layer_params(s, ix, l, t, T, True):
                w.dense(f"t{r}.layers.{l}.{nm}", r, dtype, p)
    for t in range(T):
        r = (P - 1) * T + t
        w.dense(f"t{r}.final_norm", r, dtype, _whole(ix, "final_norm", 1, s.H))
        w.dense(f"t{r}.output_layer", r, dtype, _rowblock(ix, "lm_head", s.V, s.H, t, T))
    lay.freeze()

    def groups() -> Iterator[LoaderGroup]:
        yield [ix["embed_tokens"]], lambda ts: {
            f"t{t}.word_embeddings": c for t, c in enumerate(ts[0].chunk(T, 0))}
        for l in range(s.L):
            def layer(ts, l=l):
                pp = l // per_stage
                out = {}
                for t in range(T):
                    for nm, x in _mega_layer_tensors(s, ts, t, T, True):
                        out[f"t{pp * T + t}.layers.{l}.{nm}"] = x
                return out
            yield [ix[f"layers.{l}.{n}"] for n in _DENSE_LAYER], layer

        def final(ts):
            out = {}
            for t in range(T):
                r = (P - 1) * T + t
                out[f"t{r}.final_norm"] = ts[0].clone()
                out[f"t{r}.output_layer"] = ts[1].chunk(T, 0)[t]
            return out
        yield [ix["final_norm"], ix["lm_head"]], final
    return lay, groups


# --------------------------------------------------------------------------------------
# rollout layouts
# --------------------------------------------------------------------------------------
def rollout_tp(s: ModelSpec, ck, ix, R: int, dtype: int):
    """Inference layout with TP=R: fused qkv_proj / gate_up_proj, column-split o_proj and
    down_proj, vocab-split embeddings, norms on every rank; MoE experts stacked (EP=1)."""
    lay = Layout("rollout")
    w = _SliceWriter(lay, ck)
    for r in range(R):
        w.dense(f"r{r}.embed_tokens", r, dtype, _rowblock(ix, "embed_tokens", s.V, s.H, r, R))
    for l in range(s.L):
        p = f"layers.{l}."
        for r in range(R):
            qr, kr = s.nq * s.hd // R, s.nkv * s.hd // R
            w.dense(f"r{r}.{p}qkv_proj", r, dtype, Param(qr + 2 * kr, s.H, [
                (0, qr, ix[p + "q_proj"], r * qr, 0),
                (qr, kr, ix[p + "k_proj"], r * kr, 0),
                (qr + kr, kr, ix[p + "v_proj"], r * kr, 0)]))
            w.dense(f"r{r}.{p}o_proj", r, dtype, _colblock(ix, p + "o_proj", s.H, s.nq * s.hd, r, R))
            if s.E:
                assert R == 1
                w.dense(f"r{r}.{p}router", r, dtype, _whole(ix, p + "router", s.E, s.H))
                b13, b2 = [], []
                for e in range(s.E):
                    b13.append((e * 2 * s.Fe, s.Fe, ix[p + f"experts.{e}.gate_proj"], 0, 0))
                    b13.append((e * 2 * s.Fe + s.Fe, s.Fe, ix[p + f"experts.{e}.up_proj"], 0, 0))
                    b2.append((e * s.H, s.H, ix[p + f"experts.{e}.down_proj"], 0, 0))
                w.dense(f"r{r}.{p}w13", r, dtype, Param(s.E * 2 * s.Fe, s.H, b13))
                w.dense(f"r{r}.{p}w2", r, dtype, Param(s.E * s.H, s.Fe, b2))
            else:
                Fr = s.F // R
                w.dense(f"r{r}.{p}gate_up_proj", r, dtype, Param(2 * Fr, s.H, [
                    (0, Fr, ix[p + "gate_proj"], r * Fr, 0),
                    (Fr, Fr, ix[p + "up_proj"], r * Fr, 0)]))
                w.dense(f"r{r}.{p}down_proj", r, dtype, _colblock(ix, p + "down_proj", s.H, s.F, r, R))
            w.dense(f"r{r}.{p}input_norm", r, dtype, _whole(ix, p + "input_norm", 1, s.H))
            w.dense(f"r{r}.{p}post_attn_norm", r, dtype, _whole(ix, p + "post_attn_norm", 1, s.H))
    for r in range(R):
        w.dense(f"r{r}.final_norm", r, dtype, _whole(ix, "final_norm", 1, s.H))
        w.dense(f"r{r}.lm_head", r, dtype, _rowblock(ix, "lm_head", s.V, s.H, r, R))
    lay.freeze()

    def groups() -> Iterator[LoaderGroup]:
        yield [ix["embed_tokens"]], lambda ts: {
            f"r{r}.embed_tokens": c for r, c in enumerate(ts[0].chunk(R, 0))}
        for l in range(s.L):
            p = f"layers.{l}."

            def attn(ts, p=p):
                q, k, v, o, n1, n2 = ts
                out = {}
                for r in range(R):
                    out[f"r{r}.{p}qkv_proj"] = torch.cat(
                        [q.chunk(R, 0)[r], k.chunk(R, 0)[r], v.chunk(R, 0)[r]], 0)
                    out[f"r{r}.{p}o_proj"] = o.chunk(R, 1)[r]
                    out[f"r{r}.{p}input_norm"] = n1.clone()
                    out[f"r{r}.{p}post_attn_norm"] = n2.clone()
                return out
            yield [ix[p + n] for n in ("q_proj", "k_proj", "v_proj", "o_proj",
                                       "input_norm", "post_attn_norm")], attn
            if s.E:
                yield [ix[p + "router"]], lambda ts, p=p: {f"r0.{p}router": ts[0]}

                def w13(ts, p=p):
                    g, u = ts[:s.E], ts[s.E:]
                    return {f"r0.{p}w13": torch.stack(
                        [torch.cat([g[e], u[e]], 0) for e in range(s.E)], 0)}
                yield ([ix[p + f"experts.{e}.gate_proj"] for e in range(s.E)] +
                       [ix[p + f"experts.{e}.up_proj"] for e in range(s.E)]), w13
                yield [ix[p + f"experts.{e}.down_proj"] for e in range(s.E)], \
                    lambda ts, p=p: {f"r0.{p}w2": torch.stack(ts, 0)}
            else:
                def mlp(ts, p=p):
                    gate, up, down = ts
                    out = {}
                    for r in range(R):
                        out[f"r{r}.{p}gate_up_proj"] = torch.cat(
                            [gate.chunk(R, 0)[r], up.chunk(R, 0)[r]], 0)
                        out[f"r{r}.{p}down_proj"] = down.chunk(R, 1)[r]
                    return out
                yield [ix[p + n] for n in ("gate_proj", "up_proj", "down_proj")], mlp

        def final(ts):
            out = {}
            for r in range(R):
                out[f"r{r}.final_norm"] = ts[0].clone()
                out[f"r{r}.lm_head"] = ts[1].chunk(R, 0)[r]
            return out
        yield [ix["final_norm"], ix["lm_head"]], final
    return lay, groups


# --------------------------------------------------------------------------------------
# stress workload: many small tensors, random shardings
# --------------------------------------------------------------------------------------
def _chunk_bounds(n: int, k: int) -> List[Tuple[int, int]]:
    """torch.chunk semantics: size ceil(n/k), ceil(n/size) parts, trailing ranks empty."""
    size = -(-n // k)
    return [(b, min(b + size, n)) for b in range(0, n, size)]


def stress_workload(n_tensors: int, dim_lo: int, dim_ratio: float, cap_bytes: int, seed: int,
                    src_dtype: int, dst_dtype: int):
    rng = SplitMix64(seed)
    ck: List[CkptTensor] = []
    recipe = []
    kinds = ("row", "col", "flat")
    for i in range(n_tensors):
        while True:
            rows = int(dim_lo * dim_ratio ** rng.uniform())
            cols = int(dim_lo * dim_ratio ** rng.uniform())
            if rows * cols * 4 <= cap_bytes:
                break
        tk = rng.randint(0, 2)
        tparts = rng.randint(2, 8)
        rk = [k for k in range(3) if k != tk][rng.randint(0, 1)]
        rparts = [p for p in range(2, 9) if p != tparts][rng.randint(0, 5)]
        transposed = rng.uniform() < 0.3
        ck.append(CkptTensor(f"s{i}", rows, cols))
        recipe.append((kinds[tk], tparts, kinds[rk], rparts, transposed))

    def build_side(side: str, dtype: int) -> Layout:
        lay = Layout(side)
        pre = "t" if side == "trainer" else "r"
        for i, c in enumerate(ck):
            tkind, tparts, rkind, rparts, tr = recipe[i]
            kind, parts = (tkind, tparts) if side == "trainer" else (rkind, rparts)
            tr = tr and side == "rollout"
            if kind == "row":
                for k, (b, e) in enumerate(_chunk_bounds(c.rows, parts)):
                    t = lay.add_tensor(f"{pre}{k}.s{i}", k, dtype, (e - b) * c.cols)
                    sr, sc = (1, e - b) if tr else (c.cols, 1)
                    lay.add_slice(t, 0, sr, sc, i, c.rows, c.cols, b, 0, e - b, c.cols)
            elif kind == "col":
                for k, (b, e) in enumerate(_chunk_bounds(c.cols, parts)):
                    t = lay.add_tensor(f"{pre}{k}.s{i}", k, dtype, c.rows * (e - b))
                    sr, sc = (1, c.rows) if tr else (e - b, 1)
                    lay.add_slice(t, 0, sr, sc, i, c.rows, c.cols, 0, b, c.rows, e - b)
            else:
                # flat split of the stored matrix: the checkpoint matrix itself, or (when
                # transposed) its transpose [cols, rows]
                width = c.rows if tr else c.cols
                for k, (b, e) in enumerate(_chunk_bounds(c.numel, parts)):
                    t = lay.add_tensor(f"{pre}{k}.s{i}", k, dtype, e - b)
                    for (a0, b0, na, nb, fstart) in flat_range_rects(width, b, e):
                        if tr:   # (a, b) index the transpose: a over ckpt cols, b over ckpt rows
                            lay.add_slice(t, fstart - b, 1, c.rows, i, c.rows, c.cols, b0, a0, nb, na)
                        else:
                            lay.add_slice(t, fstart - b, c.cols, 1, i, c.rows, c.cols, a0, b0, na, nb)
        return lay.freeze()

    def groups_for(side: str):
        pre = "t" if side == "trainer" else "r"

        def groups() -> Iterator[LoaderGroup]:
            for i in range(n_tensors):
                tkind, tparts, rkind, rparts, tr = recipe[i]
                kind, parts = (tkind, tparts) if side == "trainer" else (rkind, rparts)
                tr = tr and side == "rollout"

                def fn(ts, i=i, kind=kind, parts=parts, tr=tr):
                    A = ts[0]
                    if kind == "flat":
                        M = A.t().contiguous() if tr else A
                        ps = M.reshape(-1).chunk(parts)
                    else:
                        ps = A.chunk(parts, 0 if kind == "row" else 1)
                        if tr:
                            ps = [p.t() for p in ps]
                    return {f"{pre}{k}.s{i}": p.contiguous() for k, p in enumerate(ps)}
                yield [i], fn
        return groups

    return ck, recipe, build_side("trainer", src_dtype), build_side("rollout", dst_dtype), \
        groups_for("trainer"), groups_for("rollout")


# --------------------------------------------------------------------------------------
# the named configurations
# --------------------------------------------------------------------------------------
_TINY = ModelSpec(L=2, H=256, nq=4, nkv=2, hd=64, F=688, V=1024)
_SHAPES = {
    # config: {scale: spec}
    "cfg2": {"full": ModelSpec(32, 4096, 32, 8, 128, 14336, 128256),
             "large": ModelSpec(4, 4096, 32, 8, 128, 14336, 16032),      # ~2 GB per side
             "medium": ModelSpec(2, 1024, 16, 4, 64, 3576, 8200),
             "small": ModelSpec(2, 256, 8, 2, 32, 696, 1000)},
    "cfg3": {"full": ModelSpec(32, 4096, 32, 8, 128, 14336, 128256),
             "large": ModelSpec(4, 4096, 32, 8, 128, 14336, 16032),
             "medium": ModelSpec(4, 1024, 16, 8, 64, 3584, 8192),
             "small": ModelSpec(4, 256, 8, 4, 32, 704, 1024)},
    "cfg4": {"full": ModelSpec(48, 2048, 32, 4, 128, 0, 151936, E=128, Fe=768),
             "large": ModelSpec(2, 2048, 32, 4, 128, 0, 16032, E=128, Fe=768),
             "medium": ModelSpec(2, 512, 8, 2, 64, 0, 8200, E=32, Fe=192),
             "small": ModelSpec(2, 128, 8, 2, 32, 0, 1000, E=16, Fe=48)},
}
_STRESS = {"full": (4000, 16, 512.0, 1 << 26),
           "large": (500, 16, 512.0, 1 << 26),
           "medium": (600, 8, 256.0, 1 << 22),
           "small": (300, 4, 64.0, 1 << 20)}


def make_workload(name: str, scale: str = "full") -> Workload:
    """Build a named configuration.  `scale` is 'full' (the benchmark shape), 'large' (the
    same shapes with fewer layers / tensors, a few GB: larger than L2 but small enough for a
    profiler capture), or a shrunken 'medium' / 'small' copy of the same layout family for
    parity tests
    (cfg1, cfg1b and cfg1c are already tiny and ignore it)."""
    if name in ("cfg1", "cfg1b", "cfg1c"):
        s = _TINY
        ck, ix = build_ckpt(s)
        W = 3 if name == "cfg1b" else 2
        tl, tg = trainer_tp_fsdp(s, ck, ix, T=2, W=W, dtype=WB_F32, fused=(name != "cfg1c"))
        rl, rg = rollout_tp(s, ck, ix, R=1, dtype=WB_BF16)
        return Workload(name, 0, "normal0.02", WB_F32, WB_BF16, ck, tl, rl, tg, rg,
                        meta={"spec": s, "distinct_read_elems": sum(c.numel for c in ck)})
    if name == "cfg2":
        s = _SHAPES[name][scale]
        ck, ix = build_ckpt(s)
        tl, tg = trainer_fsdp(s, ck, ix, W=8, dtype=WB_BF16)
        rl, rg = rollout_tp(s, ck, ix, R=1, dtype=WB_BF16)
        return Workload(f"{name}-{scale}", 1, "normal0.02", WB_BF16, WB_BF16, ck, tl, rl, tg, rg,
                        meta={"spec": s, "distinct_read_elems": sum(c.numel for c in ck)})
    if name == "cfg3":
        s = _SHAPES[name][scale]
        ck, ix = build_ckpt(s)
        tl, tg = trainer_tp_pp(s, ck, ix, T=4, P=2, dtype=WB_F32)
        rl, rg = rollout_tp(s, ck, ix, R=2, dtype=WB_BF16)
        return Workload(f"{name}-{scale}", 2, "normal0.02", WB_F32, WB_BF16, ck, tl, rl, tg, rg,
                        meta={"spec": s, "distinct_read_elems": sum(c.numel for c in ck)})
    if name == "cfg4":
        s = _SHAPES[name][scale]
        ck, ix = build_ckpt(s)
        tl, tg = trainer_fsdp(s, ck, ix, W=8, dtype=WB_BF16, EP=8)
        rl, rg = rollout_tp(s, ck, ix, R=1, dtype=WB_BF16)
        return Workload(f"{name}-{scale}", 3, "normal0.02", WB_BF16, WB_BF16, ck, tl, rl, tg, rg,
                        meta={"spec": s, "distinct_read_elems": sum(c.numel for c in ck)})
    if name == "cfg5":
        n, lo, ratio, cap = _STRESS[scale]
        ck, recipe, tl, rl, tg, rg = stress_workload(n, lo, ratio, cap, 4, WB_F32, WB_BF16)
        return Workload(f"{name}-{scale}", 4, "uniform", WB_F32, WB_BF16, ck, tl, rl, tg, rg,
                        meta={"recipe": recipe, "distinct_read_elems": sum(c.numel for c in ck)})
    raise ValueError(name)
