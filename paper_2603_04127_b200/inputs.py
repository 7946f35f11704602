"""Seeded synthetic inputs for the DARK-attention workloads.

This module only draws random tensors (anisotropic Gaussian queries/keys, Gaussian values,
near-identity geometry matrices, Gaussian projection rows) and rounds them to a storage type.
It contains none of the attention arithmetic, so both the CUDA path and the CPU oracle may be
fed from it without sharing any of the method's code.

Everything is generated in float64 with one ``numpy.random.default_rng(seed)`` stream per tensor.
"""
from __future__ import annotations

from dataclasses import dataclass, field
import numpy as np

# index of each tensor's random stream inside a workload (seed = 1000 * workload_id + index)
_STREAMS = {"U": 0, "Q": 1, "K": 2, "V": 3, "G": 4, "W": 5, "dO": 6}


@dataclass(frozen=True)
class Workload:
    """Shape and distribution parameters of one synthetic workload."""
    name: str
    wid: int                 # workload id, selects the seeds
    B: int
    H: int
    N: int
    d: int
    m: int
    dtype: str               # "f32" or "bf16": storage type of Q,K,V,M,W,O
    causal: bool
    backward: bool = False
    rho: float = 0.9         # eigenvalue decay of the query/key covariance
    top_scale: float = 1.0   # extra factor on the largest eigenvalue (after trace normalisation)
    r: int = 0               # rows of M; 0 means r = d
    dv: int = 0              # value width; 0 means dv = d

    def dims(self):
        r = self.r or self.d
        dv = self.dv or self.d
        return self.B, self.H, self.N, self.d, r, self.m, dv


# The five benchmark configurations plus the headline shape (config-3 shape with backward).
WORKLOADS = {
    "c1": Workload("c1", 1, 1, 1, 256, 64, 64, "f32", False),
    "c2": Workload("c2", 2, 8, 12, 4096, 64, 256, "bf16", False),
    "c3": Workload("c3", 3, 4, 16, 8192, 128, 256, "bf16", True, rho=0.95),
    "c4": Workload("c4", 4, 1, 8, 65536, 64, 512, "bf16", True, top_scale=4.0),
    "c5": Workload("c5", 5, 8, 12, 2048, 64, 256, "bf16", True, backward=True),
    "headline": Workload("headline", 3, 4, 16, 8192, 128, 256, "bf16", True, backward=True, rho=0.95),
    # the headline shape without the causal mask (bidirectional attention), forward + backward
    "headline_nc": Workload("headline_nc", 6, 4, 16, 8192, 128, 256, "bf16", False, backward=True, rho=0.95),
}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64/float32 values to the nearest bfloat16 (ties to even); returns float32 values."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    out = ((u + bias) & np.uint32(0xFFFF0000)).view(np.float32)
    return out.reshape(f.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Upper 16 bits (the bfloat16 pattern) of float32 values that are already bf16-representable."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    return (f.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(f.shape)


def covariance_spectrum(d: int, rho: float, top_scale: float = 1.0) -> np.ndarray:
    """lambda_i = rho**i scaled so that sum(lambda) = d; then lambda_0 *= top_scale."""
    lam = rho ** np.arange(d, dtype=np.float64)
    lam *= d / lam.sum()
    lam[0] *= top_scale
    return lam


def random_orthogonal(d: int, rng: np.random.Generator) -> np.ndarray:
    """QR of a Gaussian matrix with the column signs fixed by sign(diag R)."""
    a = rng.standard_normal((d, d))
    q, rr = np.linalg.qr(a)
    return q * np.sign(np.diag(rr))[None, :]


def orthogonal_projection_rows(m: int, r: int, rng: np.random.Generator) -> np.ndarray:
    """W [m, r] in blocks of r rows: each block is a Haar-random orthogonal basis whose rows are rescaled to the
    norms of independent N(0, I_r) vectors, so every row is marginally N(0, I_r) while the rows of a block are
    exactly orthogonal (the orthogonal random features Section 2 mentions). Blocks are independent."""
    blocks = []
    for _ in range((m + r - 1) // r):
        q = random_orthogonal(r, rng)
        norms = np.linalg.norm(rng.standard_normal((r, r)), axis=1)
        blocks.append(q * norms[:, None])
    return np.concatenate(blocks, axis=0)[:m]


def optimal_proposal_spectrum(lam: np.ndarray) -> np.ndarray:
    """Eigenvalues of Sigma* = (I + 2 Lambda)(I - 2 Lambda)^-1 (Theorem 3.2) for the eigenvalues ``lam`` of the
    input covariance Lambda; a valid covariance only while max(lam) < 1/2."""
    lam = np.asarray(lam, dtype=np.float64)
    if not (lam.max() < 0.5 and lam.min() >= 0.0):
        raise ValueError("Sigma* is a covariance only for 0 <= lambda < 1/2")
    return (1.0 + 2.0 * lam) / (1.0 - 2.0 * lam)


def aligned_M(U: np.ndarray, lam: np.ndarray) -> np.ndarray:
    """M [d, d] with M^T M = U diag(sigma*) U^T, sigma* = optimal_proposal_spectrum(lam): the geometry of the
    variance-optimal Gaussian proposal for inputs of covariance U diag(lam) U^T."""
    return np.sqrt(optimal_proposal_spectrum(lam))[:, None] * U.T


def variance_workload(wid: int, B: int, H: int, N: int, d: int, m: int, lam_max: float = 0.2, aligned: bool = True,
                      causal: bool = False, dtype: str = "bf16", backward: bool = True, dv: int = 0) -> "Tensors":
    """The second synthetic workload: Gaussian queries and keys of covariance Lambda = U diag(lam) U^T with a
    geometric spectrum below 1/2 (lam_i = lam_max * 0.9**i), orthogonal projection rows W, and M either the
    identity (isotropic sampling) or aligned_M(U, lam) (data-aligned sampling, the same for every head). Use it
    with scale = 1."""
    wl = Workload(f"variance_{'aligned' if aligned else 'isotropic'}", wid, B, H, N, d, m, dtype, causal, backward, 0.9, 1.0, 0, dv)
    _, _, _, _, r, _, dvv = wl.dims()
    U = random_orthogonal(d, _rng(wid, "U"))
    lam = lam_max * 0.9 ** np.arange(d, dtype=np.float64)
    draw = lambda stream, width, aniso: np.stack([
        (anisotropic_rows(wid, stream, N, U, lam, b * H + h) if aniso else _rng(wid, stream, b * H + h).standard_normal((N, width)))
        for b in range(B) for h in range(H)]).reshape(B, H, N, width)
    Q, K, V = draw("Q", d, True), draw("K", d, True), draw("V", dvv, False)
    dO = draw("dO", dvv, False) if backward else None
    M = np.broadcast_to((aligned_M(U, lam) if aligned else np.eye(d))[None], (H, d, d)).copy()
    W = orthogonal_projection_rows(m, r, _rng(wid, "W"))
    if dtype == "bf16":
        rt = lambda a: None if a is None else round_to_bf16(a).astype(np.float64)
    else:
        rt = lambda a: None if a is None else a.astype(np.float32).astype(np.float64)
    return Tensors(wl, rt(Q), rt(K), rt(V), rt(M), rt(W), rt(dO), [(b, h) for b in range(B) for h in range(H)])


def _rng(wid: int, stream: str, extra: int = 0) -> np.random.Generator:
    return np.random.default_rng([1000 * wid + _STREAMS[stream], extra])


def anisotropic_rows(wid: int, stream: str, n_rows: int, U: np.ndarray, lam: np.ndarray,
                     block: int = 0) -> np.ndarray:
    """n_rows draws of U diag(sqrt(lam)) g with g ~ N(0, I)."""
    g = _rng(wid, stream, block).standard_normal((n_rows, U.shape[0]))
    return (g * np.sqrt(lam)[None, :]) @ U.T


@dataclass
class Tensors:
    """Float64 tensors of one workload (already rounded to the storage type where that is bf16)."""
    wl: Workload
    Q: np.ndarray
    K: np.ndarray
    V: np.ndarray
    M: np.ndarray
    W: np.ndarray
    dO: np.ndarray | None
    heads: list = field(default_factory=list)   # the (b, h) pairs held, in order, when subsampled


def generate(wl: Workload, pairs=None, as_batch: bool = False) -> Tensors:
    """Generate the tensors of a workload.

    Each (b, h) slice has its own random stream, so a subset of pairs (``pairs`` = list of (b, h))
    reproduces exactly the values the full tensor has at those positions. With ``pairs=None`` the
    full [B,H,N,*] tensors are returned. Otherwise the requested slices are returned in order as a
    problem of their own: by default with shapes [1, P, N, *] (each pair a head, M gathered to
    [P, r, d]); with ``as_batch`` (all pairs must name the same head h) with shapes [P, 1, N, *] and
    M = M[h:h+1], so that a gradient of M sums over the pairs exactly as it sums over the batch.
    """
    B, H, N, d, r, m, dv = wl.dims()
    U = random_orthogonal(d, _rng(wl.wid, "U"))
    lam = covariance_spectrum(d, wl.rho, wl.top_scale)
    all_pairs = [(b, h) for b in range(B) for h in range(H)]
    use = all_pairs if pairs is None else list(pairs)

    def draw(stream, width, aniso):
        out = np.empty((len(use), N, width), dtype=np.float64)
        for i, (b, h) in enumerate(use):
            blk = b * H + h
            if aniso:
                out[i] = anisotropic_rows(wl.wid, stream, N, U, lam, blk)
            else:
                out[i] = _rng(wl.wid, stream, blk).standard_normal((N, width))
        return out

    Q = draw("Q", d, True)
    K = draw("K", d, True)
    V = draw("V", dv, False)
    dO = draw("dO", dv, False) if wl.backward else None
    G = _rng(wl.wid, "G").standard_normal((H, r, d)) / np.sqrt(d)
    M = np.eye(r, d)[None, :, :] + 0.1 * G
    W = _rng(wl.wid, "W").standard_normal((m, r))

    if pairs is None:
        shp = lambda w: (B, H, N, w)
    elif as_batch:
        hs = {h for _, h in use}
        assert len(hs) == 1, "as_batch needs pairs of one head"
        shp = lambda w: (len(use), 1, N, w)
        M = M[[next(iter(hs))]]
    else:
        shp = lambda w: (1, len(use), N, w)
        M = M[[h for _, h in use]]
    Q, K, V = Q.reshape(shp(d)), K.reshape(shp(d)), V.reshape(shp(dv))
    if dO is not None:
        dO = dO.reshape(shp(dv))
    if wl.dtype == "bf16":
        rt = lambda a: None if a is None else round_to_bf16(a).astype(np.float64)
        Q, K, V, M, W, dO = rt(Q), rt(K), rt(V), rt(M), rt(W), rt(dO)
    elif wl.dtype == "f32":
        rt = lambda a: None if a is None else a.astype(np.float32).astype(np.float64)
        Q, K, V, M, W, dO = rt(Q), rt(K), rt(V), rt(M), rt(W), rt(dO)
    return Tensors(wl, Q, K, V, M, W, dO, use)


def parameters(wl: Workload):
    """The parameters M [H, r, d] and W [m, r] of a workload alone (the same values generate() returns), rounded to the
    workload's storage type: what every rank of a data-parallel job shares while it draws its own batch."""
    B, H, N, d, r, m, dv = wl.dims()
    G = _rng(wl.wid, "G").standard_normal((H, r, d)) / np.sqrt(d)
    M = np.eye(r, d)[None, :, :] + 0.1 * G
    W = _rng(wl.wid, "W").standard_normal((m, r))
    if wl.dtype == "bf16":
        return round_to_bf16(M).astype(np.float64), round_to_bf16(W).astype(np.float64)
    return M.astype(np.float32).astype(np.float64), W.astype(np.float32).astype(np.float64)


def small(name="tiny", wid=9, B=1, H=2, N=16, d=8, m=16, causal=False, dtype="f32", backward=True,
          rho=0.9, r=0, dv=0, top_scale=1.0) -> Workload:
    """A free-form small workload for tests."""
    return Workload(name, wid, B, H, N, d, m, dtype, causal, backward, rho, top_scale, r, dv)
