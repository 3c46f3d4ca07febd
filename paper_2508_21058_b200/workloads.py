"""Seeded synthetic workloads: token layouts and Q/K/V/dO generators.

This module serves both the CUDA library's tests/bench and the CPU oracle's tests.
It holds none of the method's arithmetic (no pooling, scoring, selection or
attention): only integer layout tables and a counter-based random generator.

Layouts stand in for the paper's token streams (Sec. 3.2 "Content-aligned
Chunking"; the Wan-2.1 experiment's 1560 tokens per latent frame; the multi-shot
setting of interleaved caption + shot tokens).  Every value is a pure function of
(seed, tensor id, head, token, dim), so the same bf16 bit patterns come out on the
CPU and on a GPU:

  * a 32-bit integer mixer is evaluated with int64 tensor ops whose intermediate
    products stay below 2**63 (no reliance on overflow wrap-around);
  * standard-normal variates come from a 65536-entry inverse-CDF table built once
    on the host in float64 and rounded to float32, indexed by 16 hash bits;
  * the only floating-point steps are ``0.5 * centre`` (exact), one float32 add and
    the round-to-nearest-even cast to bf16, all correctly rounded on both devices.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from functools import lru_cache

import numpy as np
import torch

_M32 = 0xFFFFFFFF

# tensor ids of the counter-based generator
_T_CENTRE, _T_K, _T_Q, _T_V, _T_DO, _T_TARGET = 1, 2, 3, 4, 5, 6

WHOLE_SHOT = -1


# ----------------------------------------------------------------------------- layouts
@dataclass
class Layout:
    """Chunk table of one token stream (host numpy arrays)."""

    chunk_off: np.ndarray   # int32 [C+1]
    chunk_shot: np.ndarray  # int32 [C]
    chunk_mod: np.ndarray   # uint8 [C]  0 = video, 1 = text

    @property
    def n_chunks(self) -> int:
        return int(self.chunk_shot.shape[0])

    @property
    def n_tokens(self) -> int:
        return int(self.chunk_off[-1])

    def token_chunk(self) -> np.ndarray:
        """int32 [L]: index of the chunk that holds each token."""
        sizes = np.diff(self.chunk_off)
        return np.repeat(np.arange(self.n_chunks, dtype=np.int32), sizes)


def make_layout(n_shots: int, caption_len: int, frames_per_shot: int, frame_len: int,
                chunk_len: int | None = None) -> Layout:
    """Interleaved stream: per shot one caption (a single text chunk) followed by
    ``frames_per_shot * frame_len`` video tokens.  With ``chunk_len=None`` a video
    chunk is one frame; otherwise the shot's video tokens are cut into windows of
    ``chunk_len`` tokens restarted at every shot/modality boundary, the last one
    short."""
    off, shot, mod = [0], [], []
    for s in range(n_shots):
        if caption_len > 0:
            off.append(off[-1] + caption_len)
            shot.append(s)
            mod.append(1)
        video = frames_per_shot * frame_len
        step = frame_len if chunk_len is None else chunk_len
        done = 0
        while done < video:
            n = min(step, video - done)
            off.append(off[-1] + n)
            shot.append(s)
            mod.append(0)
            done += n
    return Layout(np.asarray(off, np.int32), np.asarray(shot, np.int32), np.asarray(mod, np.uint8))


@dataclass
class Workload:
    name: str
    n_heads: int
    head_dim: int
    layout: Layout
    top_k: int
    win_back: int
    win_fwd: int
    causal: bool = True
    seed: int = 0
    shared_identities: int = 0   # >0: each key centre is reused in this many shots
    note: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def n_tokens(self) -> int:
        return self.layout.n_tokens

    @property
    def n_chunks(self) -> int:
        return self.layout.n_chunks


def sweep_top_k(p: float, n_tokens: int, chunk_len: int, caption_tokens: int) -> int:
    """k such that selected keys are about ``p`` of the mean causal context L/2:
    anchors are all captions plus a 3-chunk window, the rest is routed."""
    return max(1, int(round((p * n_tokens / 2 - caption_tokens - 3 * chunk_len) / chunk_len)))


def workload(name: str, seed: int = 0) -> Workload:
    """Named workloads.  cfg0..cfg4 follow the benchmark configurations; the
    ``mini*`` ones are scaled-down layouts with the same structure (ragged frame
    length, several shots, captions) that the CPU oracle finishes in seconds."""
    if name == "cfg0":
        return Workload(name, 4, 64, make_layout(1, 64, 8, 64), 2, 0, 0, seed=seed,
                        note="64 text + 8 frames x 64 tokens")
    if name == "cfg1":
        return Workload(name, 24, 128, make_layout(1, 256, 21, 1560), 4, 0, 0, seed=seed,
                        note="256 text + 21 frames x 1560 tokens")
    if name == "cfg2":
        return Workload(name, 24, 128, make_layout(8, 256, 21, 1560), 6, 1, 1, seed=seed,
                        note="8 shots x (256 caption + 21 x 1560)")
    if name == "cfg4":
        return Workload(name, 24, 128, make_layout(16, 256, 21, 1560), 8, 1, 1, seed=seed,
                        note="16 shots x (256 caption + 21 x 1560), fwd + bwd")
    if name.startswith("cfg3"):
        # cfg3-m<chunk>-p<percent>, e.g. cfg3-m512-p15
        parts = dict((p[0], int(p[1:])) for p in name.split("-")[1:])
        m, pct = parts.get("m", 1560), parts.get("p", 15)
        lay = make_layout(8, 256, 21, 1560, chunk_len=m)
        k = sweep_top_k(pct / 100.0, lay.n_tokens, m, 8 * 256)
        return Workload(name, 24, 128, lay, k, 1, 1, seed=seed, shared_identities=4,
                        note=f"cfg2 tokens, chunk {m}, k={k} (~{pct}% of causal context)")
    if name == "mini1":   # single shot, ragged frames, d=128
        return Workload(name, 3, 128, make_layout(1, 48, 7, 200), 3, 0, 0, seed=seed)
    if name == "mini2":   # multi shot, window (1,1), captions of later shots are anchors
        return Workload(name, 3, 128, make_layout(3, 40, 5, 200), 3, 1, 1, seed=seed)
    if name == "mini2t":  # trailing-window reading (2,0) of the intra-shot anchor
        return Workload(name, 2, 128, make_layout(3, 40, 5, 200), 3, 2, 0, seed=seed)
    if name == "mini3":   # sweep-like: fixed windows with short tails, shared identities
        return Workload(name, 2, 128, make_layout(4, 24, 3, 300, chunk_len=128), 5, 1, 1,
                        seed=seed, shared_identities=4)
    if name == "mini4":   # whole-shot anchor (the paper's multi-shot definition), d=64
        return Workload(name, 2, 64, make_layout(3, 32, 4, 96), 2, WHOLE_SHOT, WHOLE_SHOT, seed=seed)
    if name == "mini5":   # non-causal single-shot variant: chunk 256, k=3, self + prompt
        return Workload(name, 2, 64, make_layout(1, 77, 1, 1500, chunk_len=256), 3, 0, 0,
                        causal=False, seed=seed)
    if name == "mini6":   # many small chunks, k = 12: the 16-entry pick list, two selection groups
        return Workload(name, 2, 128, make_layout(3, 16, 40, 24), 12, 1, 1, seed=seed)
    if name == "mini7":   # k = 70 of up to 122 candidates, d = 64: two selection passes of 64 picks, streamed descriptor blocks
        return Workload(name, 2, 64, make_layout(3, 16, 80, 16), 70, 1, 1, seed=seed)
    if name == "mini8":   # few chunks (one scoring operand for the three descriptor terms) with k above 4
        return Workload(name, 2, 128, make_layout(2, 32, 10, 160), 6, 1, 1, seed=seed)
    if name == "mini9":   # more than 32 chunks with k <= 4: the selection by extraction rounds, short list
        return Workload(name, 2, 64, make_layout(3, 16, 14, 96), 4, 1, 1, seed=seed)
    if name == "mini10":  # k = 20 of up to 80 candidates: the 32-entry pick list
        return Workload(name, 2, 128, make_layout(2, 16, 40, 32), 20, 1, 1, seed=seed)
    if name == "mini11":  # k = 40 of up to 120 candidates: the 64-entry register list, one selection group
        return Workload(name, 2, 64, make_layout(2, 16, 60, 32), 40, 1, 1, seed=seed)
    if name == "midi2":   # multi-shot with true 1560-token frames, small enough for a full oracle pass
        return Workload(name, 2, 128, make_layout(2, 256, 4, 1560), 3, 1, 1, seed=seed)
    raise KeyError(name)


# ----------------------------------------------------------------------------- generator
@lru_cache(maxsize=1)
def _normal_table_np() -> np.ndarray:
    from scipy.special import ndtri
    u = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
    return ndtri(u).astype(np.float32)


def _normal_table(device) -> torch.Tensor:
    return torch.from_numpy(_normal_table_np()).to(device)


def _mul32(x: torch.Tensor, c: int) -> torch.Tensor:
    """(x * c) mod 2**32 for int64 x in [0, 2**32) without exceeding 2**63."""
    lo = x * (c & 0xFFFF)
    hi = (x * (c >> 16)) & 0xFFFF
    return (lo + (hi << 16)) & _M32


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """32-bit integer finaliser (xor-shift-multiply rounds) on int64 storage."""
    x = x ^ (x >> 16)
    x = _mul32(x, 0x7FEB352D)
    x = x ^ (x >> 15)
    x = _mul32(x, 0x846CA68B)
    x = x ^ (x >> 16)
    return x


def _mix32_int(x: int) -> int:
    x &= _M32
    x ^= x >> 16
    x = (x * 0x7FEB352D) & _M32
    x ^= x >> 15
    x = (x * 0x846CA68B) & _M32
    x ^= x >> 16
    return x


def _stream_keys(seed: int, tensor_id: int) -> tuple[int, int]:
    k1 = _mix32_int(seed * 0x9E3779B1 + tensor_id * 0x85EBCA77 + 0x165667B1)
    k2 = _mix32_int(k1 ^ 0xC2B2AE3D)
    return k1, k2


def _hash_counter(idx: torch.Tensor, seed: int, tensor_id: int) -> torch.Tensor:
    """uint32 hash (int64 storage) of a non-negative int64 counter."""
    k1, k2 = _stream_keys(seed, tensor_id)
    h = _mix32((idx & _M32) ^ k1)
    h = _mix32((h + (idx >> 32) + k2) & _M32)
    return h


def _normals(idx: torch.Tensor, seed: int, tensor_id: int, table: torch.Tensor) -> torch.Tensor:
    return table[_hash_counter(idx, seed, tensor_id) >> 16]


def centre_ids(wl: Workload) -> np.ndarray:
    """int64 [C]: identity of the key centre of each chunk.  Without shared
    identities every chunk has its own; with ``shared_identities = r`` a pool of
    ceil(C_video / r) identities is dealt out so that each appears in up to r
    distinct shots (next free chunk slot of that shot); slots left over get
    fresh identities."""
    lay = wl.layout
    C = lay.n_chunks
    ids = np.arange(C, dtype=np.int64)
    r = wl.shared_identities
    if r <= 0:
        return ids
    rng = np.random.RandomState(1000003 + wl.seed)
    video = np.nonzero(lay.chunk_mod == 0)[0]
    shots = np.unique(lay.chunk_shot[video])
    free = {int(s): [int(c) for c in video if lay.chunk_shot[c] == s] for s in shots}
    n_pool = -(-len(video) // r)
    ids[:] = -1
    for ident in range(n_pool):
        order = rng.permutation(shots)
        placed = 0
        for s in order:
            if placed == r:
                break
            if free[int(s)]:
                ids[free[int(s)].pop(0)] = C + ident
                placed += 1
    fresh = np.nonzero(ids < 0)[0]
    ids[fresh] = fresh
    return ids


def _centres(wl: Workload, h: int, table: torch.Tensor, device) -> torch.Tensor:
    """float32 [C, d] centres of head h."""
    d = wl.head_dim
    ids = torch.from_numpy(centre_ids(wl)).to(device)
    n_id = 2 * wl.n_chunks + 1
    base = (h * n_id + ids) * d
    idx = base[:, None] + torch.arange(d, device=device, dtype=torch.int64)[None, :]
    return _normals(idx, wl.seed, _T_CENTRE, table)


def generate(wl: Workload, device="cpu", tensors=("q", "k", "v"), heads=None) -> dict[str, torch.Tensor]:
    """bf16 tensors [H, L, d] on ``device``.  Per (head, chunk) a centre
    c ~ N(0,1)^d; K_t = 0.5 c_{chunk(t)} + N(0,1); Q_i = 0.5 c_j + N(0,1) with j
    uniform over the chunks {0..chunk(i)}; V, dO ~ N(0,1)."""
    device = torch.device(device)
    H, L, d = wl.n_heads, wl.n_tokens, wl.head_dim
    heads = list(range(H)) if heads is None else list(heads)
    table = _normal_table(device)
    tok_chunk = torch.from_numpy(wl.layout.token_chunk().astype(np.int64)).to(device)
    tok = torch.arange(L, device=device, dtype=torch.int64)
    dim = torch.arange(d, device=device, dtype=torch.int64)
    out = {t: torch.empty((len(heads), L, d), dtype=torch.bfloat16, device=device) for t in tensors}
    rows = max(1, (1 << 22) // d)  # bound the int64 temporaries
    for hi, h in enumerate(heads):
        cen = _centres(wl, h, table, device) if ("q" in tensors or "k" in tensors) else None
        for r0 in range(0, L, rows):
            r1 = min(L, r0 + rows)
            t = tok[r0:r1]
            idx = ((h * L + t) * d)[:, None] + dim[None, :]
            for name in tensors:
                if name == "k":
                    val = 0.5 * cen[tok_chunk[r0:r1]] + _normals(idx, wl.seed, _T_K, table)
                elif name == "q":
                    tgt = _hash_counter(h * L + t, wl.seed, _T_TARGET) % (tok_chunk[r0:r1] + 1)
                    val = 0.5 * cen[tgt] + _normals(idx, wl.seed, _T_Q, table)
                elif name == "v":
                    val = _normals(idx, wl.seed, _T_V, table)
                elif name == "do":
                    val = _normals(idx, wl.seed, _T_DO, table)
                else:
                    raise KeyError(name)
                out[name][hi, r0:r1] = val.to(torch.bfloat16)
    return out


def as_u16(t: torch.Tensor) -> np.ndarray:
    """Host uint16 view of a bf16 tensor's bit patterns (copies to the CPU)."""
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16)


def sample_rows(wl: Workload, per_head: int, seed: int = 0) -> np.ndarray:
    """int32 [n, 2] (head, token) pairs, about ``per_head`` per head: at most half of them
    are first and last tokens of chunks (frame, caption and shot edges, which include rows
    with fewer than k candidates; a seeded subset when there are more edges than that), the
    rest are seeded uniform picks over the whole stream, so rows in the interior of every
    kind of chunk are always present whatever the number of edges."""
    lay = wl.layout
    edges = np.unique(np.concatenate([lay.chunk_off[:-1], lay.chunk_off[1:] - 1]))
    rng = np.random.RandomState(7919 + seed)
    out = []
    for h in range(wl.n_heads):
        toks = edges
        n_edge = max(1, per_head // 2)
        if len(toks) > n_edge:
            toks = np.sort(rng.choice(toks, n_edge, replace=False))
        extra = per_head - len(toks)
        if extra > 0:
            toks = np.unique(np.concatenate([toks, rng.randint(0, lay.n_tokens, extra)]))
        out.append(np.stack([np.full(len(toks), h), toks], 1))
    return np.concatenate(out).astype(np.int32)
