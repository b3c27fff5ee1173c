"""Seeded synthetic inputs for the retrieval hot path.

Everything here produces *inputs* (an index and queries); nothing here scores a
query.  The same arrays feed the CPU oracle and the CUDA library, so neither
side ever sees data the other produced.  Index construction (which inverted
list a vector joins, which codeword a residual snaps to) is part of building
the inputs and lives here, outside the search path.

Shapes follow the workloads of the RAG retrieval stage: a Gaussian-mixture
corpus whose mixture centres are the coarse centroids, product-quantised
residuals at one byte per sub-space, inverted lists stored contiguously
(CSR offsets), int64 ids, and queries drawn from the same mixture.

All tensors are torch tensors on the requested device; integer streams come
from a counter-based 64-bit mixer so any slice can be regenerated bit-exactly
on another device, floating-point streams from a seeded torch.Generator.
"""

from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional

import torch

MASTER_SEED = 0x5241474F
SIGMA = 0.3  # std of mixture noise and of codeword coordinates

_U64 = 1 << 64


def _s64(c: int) -> int:
    """Two's-complement view of a 64-bit constant as a Python int in int64 range."""
    c &= _U64 - 1
    return c - _U64 if c >= (1 << 63) else c


_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)
_GOLD = _s64(0x9E3779B97F4A7C15)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift on int64 (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def mix64(x: torch.Tensor) -> torch.Tensor:
    """Stateless 64-bit finaliser (xor-shift / multiply rounds) on int64 tensors.

    Integer-only, wraps modulo 2**64, hence bit-identical on CPU and GPU.
    """
    x = x + _GOLD
    x = (x ^ _lsr(x, 30)) * _C1
    x = (x ^ _lsr(x, 27)) * _C2
    return x ^ _lsr(x, 31)


def _stream_key(seed: int, stream: int) -> int:
    k = (seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & (_U64 - 1)
    return _s64(k)


def hash_codes(seed: int, start: int, count: int, M: int, device="cpu") -> torch.Tensor:
    """PQ codes of vectors [start, start+count) of a hash-coded index: uint8 [count, M].

    Eight consecutive code bytes are the little-endian bytes of one mixed
    64-bit word, word index = (position * M) / 8.
    """
    assert M % 8 == 0
    w = M // 8
    idx = torch.arange(start * w, (start + count) * w, dtype=torch.int64, device=device)
    h = mix64(idx ^ _stream_key(seed, 1))
    return h.view(torch.uint8).reshape(count, M)


def hash_ids(start: int, count: int, device="cpu") -> torch.Tensor:
    """ids of positions [start, start+count): a bijection of Z_2^62, so unique and >= 0."""
    pos = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return (pos * 0x2545F4914F6CDD1D + 0x1234567) & ((1 << 62) - 1)


def jitter_lengths(seed: int, N: int, nlist: int) -> torch.Tensor:
    """Deterministic list lengths within +-50% of the mean that sum to N (int64 [nlist], CPU)."""
    l = torch.arange(nlist, dtype=torch.int64)
    u = (_lsr(mix64(l ^ _stream_key(seed, 2)), 11).double() / float(1 << 53)) * 2.0 - 1.0
    raw = (1.0 + 0.5 * u)
    raw = raw / raw.sum() * N
    L = raw.floor().long()
    rem = int(N - int(L.sum()))
    L[:rem] += 1
    assert int(L.sum()) == N and int(L.min()) >= 0
    return L


def offsets_from_lengths(L: torch.Tensor) -> torch.Tensor:
    off = torch.zeros(L.numel() + 1, dtype=torch.int64)
    off[1:] = torch.cumsum(L.cpu(), 0)
    return off


def zipf_weights(n: int, s: float) -> torch.Tensor:
    r = torch.arange(1, n + 1, dtype=torch.float64)
    w = r.pow(-s)
    return w / w.sum()


@dataclass
class IvfPqData:
    """One synthetic IVF-PQ problem.  Tensors live on `device` unless noted."""

    N: int
    d: int
    nlist: int
    M: int
    metric: str  # "l2" | "ip"
    centroids: torch.Tensor  # [nlist, d] fp32, or bf16 when coarse_bf16
    codebooks: torch.Tensor  # [M, 256, d/M] fp32
    codes: Optional[torch.Tensor]  # [N, M] uint8, list-contiguous (None: hash-coded, not materialised)
    list_offsets: torch.Tensor  # [nlist+1] int64 (CPU)
    ids: Optional[torch.Tensor]  # [N] int64 (None: hash ids, not materialised)
    queries: torch.Tensor  # [nq, d] fp32
    seed: int = MASTER_SEED
    hash_coded: bool = False
    vectors: Optional[torch.Tensor] = None  # [N, d] fp32 in list order (small cases only)
    extra: dict = field(default_factory=dict)

    @property
    def coarse_bf16(self) -> bool:
        return self.centroids.dtype == torch.bfloat16


def _generator(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed & 0x7FFFFFFFFFFFFFFF)
    return g


def encode_residuals(res: torch.Tensor, codebooks: torch.Tensor, chunk: int = 8192) -> torch.Tensor:
    """Nearest-codeword code per sub-space: res [n, d] fp32 -> uint8 [n, M].

    Index construction for the synthetic corpus (ties go to whichever minimum
    torch.argmin reports; exact ties have probability zero for Gaussian data).
    """
    M, ksub, dsub = codebooks.shape
    n = res.shape[0]
    out = torch.empty((n, M), dtype=torch.uint8, device=res.device)
    cbn = (codebooks * codebooks).sum(-1)  # [M, 256]
    cbt = codebooks.transpose(1, 2).contiguous()  # [M, dsub, 256]
    for s in range(0, n, chunk):
        r = res[s:s + chunk].reshape(-1, M, dsub).permute(1, 0, 2)  # [M, c, dsub]
        score = cbn[:, None, :] - 2.0 * torch.bmm(r, cbt)  # [M, c, 256]
        out[s:s + chunk] = score.argmin(-1).t().to(torch.uint8)
    return out


def make_ivfpq(N: int, d: int, nlist: int, M: int, nq: int, *, metric: str = "l2",
               seed: int = MASTER_SEED, zipf: Optional[float] = None, assign: str = "component",
               coarse_bf16: bool = False, device="cpu", keep_vectors: bool = False,
               chunk: int = 1 << 16, shuffle_ids: bool = True) -> IvfPqData:
    """Gaussian-mixture corpus with encoded residual PQ codes.

    centres ~ N(0,1)^d are the coarse centroids; a vector is its component's
    centre plus SIGMA * N(0,1); codewords ~ N(0, SIGMA^2) per coordinate; a
    vector joins the list of its generating component (`assign="component"`)
    or of its true nearest centroid (`assign="nearest"`); its code is the
    nearest codeword of (vector - centroid) in every sub-space.  `zipf`
    gives component weights proportional to rank**-zipf (skewed list lengths),
    otherwise components are equally likely.
    """
    assert d % M == 0 and metric in ("l2", "ip")
    dev = torch.device(device)
    g = _generator(seed, dev)
    dsub = d // M
    centres = torch.randn((nlist, d), generator=g, device=dev, dtype=torch.float32)
    codebooks = SIGMA * torch.randn((M, 256, dsub), generator=g, device=dev, dtype=torch.float32)
    w = zipf_weights(nlist, zipf) if zipf else torch.full((nlist,), 1.0 / nlist, dtype=torch.float64)
    w = w.to(dev)
    comp = torch.multinomial(w.float(), N, replacement=True, generator=g) if N > 0 else \
        torch.zeros(0, dtype=torch.int64, device=dev)
    centroids_q = centres.to(torch.bfloat16) if coarse_bf16 else centres
    cen_f32 = centroids_q.float()  # the values the index actually stores

    vectors = None
    if assign == "nearest":
        x = cen_f32[comp] + SIGMA * torch.randn((N, d), generator=g, device=dev, dtype=torch.float32)
        lab = torch.empty(N, dtype=torch.int64, device=dev)
        cn = (cen_f32 * cen_f32).sum(1)
        for s in range(0, N, chunk):
            xs = x[s:s + chunk]
            lab[s:s + chunk] = (cn[None, :] - 2.0 * xs @ cen_f32.t()).argmin(1)
        order = torch.argsort(lab, stable=True)
        lab = lab[order]
        x = x[order]
        codes = encode_residuals(x - cen_f32[lab], codebooks, chunk=min(chunk, 8192))
        if keep_vectors:
            vectors = x
    else:
        lab, _ = torch.sort(comp)
        codes = torch.empty((N, M), dtype=torch.uint8, device=dev)
        if keep_vectors:
            vectors = torch.empty((N, d), dtype=torch.float32, device=dev)
        for s in range(0, N, chunk):
            c = cen_f32[lab[s:s + chunk]]
            x = c + SIGMA * torch.randn(c.shape, generator=g, device=dev, dtype=torch.float32)
            codes[s:s + chunk] = encode_residuals(x - c, codebooks, chunk=min(chunk, 8192))
            if keep_vectors:
                vectors[s:s + chunk] = x
    counts = torch.bincount(lab, minlength=nlist).cpu()
    list_offsets = offsets_from_lengths(counts)
    ids = torch.randperm(N, generator=g, device=dev) if shuffle_ids else torch.arange(N, device=dev)
    ids = ids.to(torch.int64)
    qcomp = torch.multinomial(w.float(), nq, replacement=True, generator=g)
    queries = centres[qcomp] + SIGMA * torch.randn((nq, d), generator=g, device=dev, dtype=torch.float32)
    return IvfPqData(N=N, d=d, nlist=nlist, M=M, metric=metric, centroids=centroids_q, codebooks=codebooks,
                     codes=codes, list_offsets=list_offsets, ids=ids, queries=queries, seed=seed,
                     vectors=vectors, extra={"query_component": qcomp.cpu()})


def pack_pq4(codes: torch.Tensor) -> torch.Tensor:
    """uint8 [N, M4] codes below 16 -> uint8 [N, M4/2]: sub-space 2j in the low nibble of byte j, 2j+1 in the high."""
    return (codes[:, 0::2] | (codes[:, 1::2] << 4)).contiguous()


def make_ivfpq4(N: int, d: int, nlist: int, M4: int, nq: int, *, metric: str = "l2", seed: int = MASTER_SEED,
                zipf: Optional[float] = None, coarse_bf16: bool = False, device="cpu",
                chunk: int = 1 << 16) -> IvfPqData:
    """The corpus of make_ivfpq (vectors filed under their generating component) encoded with 4-bit codes:
    M4 sub-spaces of 16 codewords ~ N(0, SIGMA^2) each, two codes per byte.  The returned record has
    M = M4 / 2 code bytes per vector, codebooks [M4, 16, d/M4] and extra["pq4"] = True."""
    assert d % M4 == 0 and M4 % 2 == 0 and metric in ("l2", "ip")
    dev = torch.device(device)
    g = _generator(seed, dev)
    centres = torch.randn((nlist, d), generator=g, device=dev, dtype=torch.float32)
    codebooks = SIGMA * torch.randn((M4, 16, d // M4), generator=g, device=dev, dtype=torch.float32)
    w = (zipf_weights(nlist, zipf) if zipf else torch.full((nlist,), 1.0 / nlist, dtype=torch.float64)).to(dev)
    comp = torch.multinomial(w.float(), N, replacement=True, generator=g) if N > 0 else \
        torch.zeros(0, dtype=torch.int64, device=dev)
    centroids_q = centres.to(torch.bfloat16) if coarse_bf16 else centres
    cen_f32 = centroids_q.float()
    lab, _ = torch.sort(comp)
    codes = torch.empty((N, M4 // 2), dtype=torch.uint8, device=dev)
    for s in range(0, N, chunk):
        c = cen_f32[lab[s:s + chunk]]
        x = c + SIGMA * torch.randn(c.shape, generator=g, device=dev, dtype=torch.float32)
        codes[s:s + chunk] = pack_pq4(encode_residuals(x - c, codebooks, chunk=min(chunk, 8192)))
    list_offsets = offsets_from_lengths(torch.bincount(lab, minlength=nlist).cpu())
    ids = torch.randperm(N, generator=g, device=dev).to(torch.int64)
    qcomp = torch.multinomial(w.float(), nq, replacement=True, generator=g)
    queries = centres[qcomp] + SIGMA * torch.randn((nq, d), generator=g, device=dev, dtype=torch.float32)
    return IvfPqData(N=N, d=d, nlist=nlist, M=M4 // 2, metric=metric, centroids=centroids_q, codebooks=codebooks,
                     codes=codes, list_offsets=list_offsets, ids=ids, queries=queries, seed=seed,
                     extra={"pq4": True, "M4": M4})


def make_ivfpq_shards(S: int, N_per: int, d: int, nlist: int, M: int, nq: int, *, metric: str = "l2",
                      seed: int = MASTER_SEED, coarse_bf16: bool = False, device="cpu") -> list:
    """S independently indexed shards of one Gaussian-mixture corpus, with one shared query batch.

    The mixture centres ~ N(0,1)^d and the queries (centre + SIGMA * N(0,1)) come from `seed`.
    Shard s draws its own N_per vectors from that mixture, its own coarse centroids (the centres
    plus 0.25 * SIGMA * N(0,1), as if it had clustered its own sample) and its own codewords, files
    a vector under its generating component and encodes the residual to that shard's centroid.
    ids are disjoint across shards: s * N_per + a permutation of [0, N_per).
    """
    assert d % M == 0 and metric in ("l2", "ip")
    dev = torch.device(device)
    g = _generator(seed, dev)
    centres = torch.randn((nlist, d), generator=g, device=dev, dtype=torch.float32)
    qcomp = torch.randint(0, nlist, (nq,), generator=g, device=dev)
    queries = centres[qcomp] + SIGMA * torch.randn((nq, d), generator=g, device=dev, dtype=torch.float32)
    shards = []
    for s in range(S):
        gs = _generator(seed + 1000003 * (s + 1), dev)
        cen = centres + 0.25 * SIGMA * torch.randn((nlist, d), generator=gs, device=dev, dtype=torch.float32)
        centroids_q = cen.to(torch.bfloat16) if coarse_bf16 else cen
        cen_f32 = centroids_q.float()
        codebooks = SIGMA * torch.randn((M, 256, d // M), generator=gs, device=dev, dtype=torch.float32)
        lab, _ = torch.sort(torch.randint(0, nlist, (N_per,), generator=gs, device=dev))
        x = centres[lab] + SIGMA * torch.randn((N_per, d), generator=gs, device=dev, dtype=torch.float32)
        codes = encode_residuals(x - cen_f32[lab], codebooks)
        ids = (torch.randperm(N_per, generator=gs, device=dev) + s * N_per).to(torch.int64)
        offsets = offsets_from_lengths(torch.bincount(lab, minlength=nlist).cpu())
        shards.append(IvfPqData(N=N_per, d=d, nlist=nlist, M=M, metric=metric, centroids=centroids_q,
                                codebooks=codebooks, codes=codes, list_offsets=offsets, ids=ids, queries=queries,
                                seed=seed, extra={"shard": s}))
    return shards


def make_coarse_tree(centroids: torch.Tensor, n1: int):
    """A second quantiser level over existing coarse centroids: node i owns the consecutive lists
    child_offsets[i] .. child_offsets[i+1]-1 (an even split of the list numbers) and its centroid is the mean of
    theirs, stored in the centroids' dtype.  Returns (level1 [n1, d], child_offsets int32 [n1 + 1], CPU)."""
    nlist = centroids.shape[0]
    assert 1 <= n1 <= nlist
    off = torch.tensor([(i * nlist) // n1 for i in range(n1 + 1)], dtype=torch.int32)
    cen = centroids.float()
    top = torch.stack([cen[int(off[i]):int(off[i + 1])].mean(0) for i in range(n1)])
    return top.to(centroids.dtype).contiguous(), off


TREE_SPREAD = 0.5  # std of a coarse centroid around its level-1 centre, when lists are drawn as a two-level hierarchy


def make_ivfpq_hashed(N: int, d: int, nlist: int, M: int, nq: int, *, metric: str, seed: int = MASTER_SEED,
                      coarse_bf16: bool = False, device="cpu", materialise: bool = True,
                      chunk: int = 1 << 22, tree_n1: Optional[int] = None) -> IvfPqData:
    """Index whose codes and ids are pure functions of (seed, position).

    Used for the shapes too large to encode from vectors: list lengths from
    `jitter_lengths`, codes from `hash_codes`, ids from `hash_ids`;
    centroids ~ N(0,1), codewords ~ N(0, SIGMA^2); a query is a random
    centroid plus SIGMA * N(0,1).  With `materialise=False` only the small
    tensors are built (a host-side caller regenerates the lists it needs).

    `tree_n1` draws the coarse centroids as a two-level hierarchy instead: tree_n1 level-1 centres
    ~ N(0,1), every list's centroid = the centre of its node (lists are dealt to nodes in equal
    consecutive runs) + TREE_SPREAD * N(0,1); extra["level1"] / extra["child_offsets"] then hold
    the second quantiser level (level-1 centroid = mean of its children, in the centroids' dtype).
    """
    dev = torch.device(device)
    g = _generator(seed, dev)
    dsub = d // M
    centres = torch.randn((nlist, d), generator=g, device=dev, dtype=torch.float32)
    if tree_n1:
        top_centres = torch.randn((tree_n1, d), generator=g, device=dev, dtype=torch.float32)
        node = (torch.arange(nlist, device=dev) * tree_n1) // nlist
        centres = top_centres[node] + TREE_SPREAD * centres
    codebooks = SIGMA * torch.randn((M, 256, dsub), generator=g, device=dev, dtype=torch.float32)
    qc = torch.randint(0, nlist, (nq,), generator=g, device=dev)
    queries = centres[qc] + SIGMA * torch.randn((nq, d), generator=g, device=dev, dtype=torch.float32)
    centroids_q = centres.to(torch.bfloat16) if coarse_bf16 else centres
    L = jitter_lengths(seed, N, nlist)
    list_offsets = offsets_from_lengths(L)
    codes = ids = None
    if materialise:
        codes = torch.empty((N, M), dtype=torch.uint8, device=dev)
        ids = torch.empty((N,), dtype=torch.int64, device=dev)
        for s in range(0, N, chunk):
            c = min(chunk, N - s)
            codes[s:s + c] = hash_codes(seed, s, c, M, dev)
            ids[s:s + c] = hash_ids(s, c, dev)
    extra = {"query_component": qc.cpu()}
    if tree_n1:
        extra["level1"], extra["child_offsets"] = make_coarse_tree(centroids_q, tree_n1)
    return IvfPqData(N=N, d=d, nlist=nlist, M=M, metric=metric, centroids=centroids_q, codebooks=codebooks,
                     codes=codes, list_offsets=list_offsets, ids=ids, queries=queries, seed=seed, hash_coded=True,
                     extra=extra)


def make_flat(N: int, d: int, nq: int, *, seed: int = MASTER_SEED, device="cpu", chunk: int = 1 << 18):
    """Flat corpus: rows ~ N(0,1)^d scaled to unit L2 norm, stored bf16; queries likewise.

    Returns (db [N, d] bf16, queries [nq, d] bf16).
    """
    dev = torch.device(device)
    g = _generator(seed ^ 0x5F1A7, dev)
    db = torch.empty((N, d), dtype=torch.bfloat16, device=dev)
    for s in range(0, N, chunk):
        c = min(chunk, N - s)
        x = torch.randn((c, d), generator=g, device=dev, dtype=torch.float32)
        db[s:s + c] = (x / x.norm(dim=1, keepdim=True)).to(torch.bfloat16)
    q = torch.randn((nq, d), generator=g, device=dev, dtype=torch.float32)
    q = (q / q.norm(dim=1, keepdim=True)).to(torch.bfloat16)
    return db, q


# The five benchmark shapes (N, d, nlist, M, nq, nprobe, k, metric, how the index is made).
CONFIGS = {
    1: dict(N=100_000, d=128, nlist=256, M=16, nq=64, nprobe=8, k=10, metric="l2", kind="encoded",
            assign="nearest", zipf=None, coarse_bf16=False),
    2: dict(N=10_000_000, d=768, nlist=4096, M=96, nq=1024, nprobe=32, k=100, metric="l2", kind="encoded",
            assign="component", zipf=1.1, coarse_bf16=False),
    3: dict(N=1_000_000_000, d=768, nlist=65_536, M=64, nq=4096, nprobe=64, k=100, metric="ip", kind="hashed",
            coarse_bf16=True),
    4: dict(N=100_000_000, d=512, nlist=16_384, M=32, nq=16, nprobe=16, k=20, metric="l2", kind="hashed",
            coarse_bf16=False),
    5: dict(N=10_000_000, d=1024, nq=256, k=100, metric="ip", kind="flat"),
}


def make_config(n: int, *, device="cpu", scale: float = 1.0, seed: int = MASTER_SEED, **over) -> IvfPqData:
    """Build benchmark shape `n` (1-4); `scale` shrinks N (and nothing else) for smaller stand-ins."""
    c = dict(CONFIGS[n])
    c.update(over)
    N = max(1, int(round(c["N"] * scale)))
    if c["kind"] == "encoded":
        return make_ivfpq(N, c["d"], c["nlist"], c["M"], c["nq"], metric=c["metric"], seed=seed, zipf=c["zipf"],
                          assign=c["assign"], coarse_bf16=c["coarse_bf16"], device=device,
                          keep_vectors=c.get("keep_vectors", False))
    if c["kind"] == "hashed":
        return make_ivfpq_hashed(N, c["d"], c["nlist"], c["M"], c["nq"], metric=c["metric"], seed=seed,
                                 coarse_bf16=c["coarse_bf16"], device=device,
                                 materialise=c.get("materialise", True), tree_n1=c.get("tree_n1"))
    raise ValueError("config %d is not an IVF-PQ shape" % n)


def batch_size_stream(seed: int, n: int = 256) -> list:
    """The iterative-retrieval stream: n batch sizes drawn from {1, 4, 16}."""
    i = torch.arange(n, dtype=torch.int64)
    h = _lsr(mix64(i ^ _stream_key(seed, 3)), 33) % 3
    return [(1, 4, 16)[int(v)] for v in h]
