"""Seeded synthetic inputs for the MtPC head (shared by the tests, the bench and the CPU oracle's callers).

This module holds NONE of the method's arithmetic: it only draws random tensors with the shapes, dtypes
and value distributions of the five workloads and quantises them to bf16 (round-to-nearest-even) so that
the CUDA path and the fp64 oracle read bit-identical values.

Workloads (stand-ins for the paper's EvaByte / Llama-byte features and trained unembeddings, which need
weights and data that are not available offline):
  0  CP tiny            T=256  d=256  n=4  r=8  v=256  fp32 io, uniform targets, + 256 draft windows
  1  CP training-shaped T=8192 d=4096 n=8  r=16 v=320  bf16, Zipf(1.1) targets
  2  HMM                T=8192 d=4096 n=8  r=32 v=320  bf16, static transitions ~N(0,1), Zipf(1.1) targets
  3  BTree              T=4096 d=3072 n=16 r=32 v=256  bf16, uniform targets, + draft wpp=1
  4  decode sweep cells P in {1,8,64}, d=4096, v=320, CP r=16 / HMM r=32, n in {8,16}, wpp=16
  5  HMM with contextual transitions: as 2, plus (n-1) r r = 7168 transition rows in W_sum and a bias ~N(0,1) + 4 I
  6  CP head shaped like the paper's byte-level Llama-3.2-3B (Table 4): d=3072, 268 symbols stored as v=272, n=8, r=16,
     fp32 io (the dtype Table 4 gives for that model)
Hidden states ~N(0,1); every weight ~N(0, std=0.02); uniforms in [0,1) as fp32. For the acceptance stage the
target model's conditionals are Dirichlet rows (target_rows) and its uniforms come from the same generator.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor

import numpy as np

CP, HMM, BTREE = 0, 1, 2
HMM_CTX = 3          # HMM with contextual transitions (C ABI: MTPC_HMM with MTPC_FLAG_HMM_CONTEXTUAL)
F32, BF16 = 0, 1
FAMILY_NAMES = {CP: "cp", HMM: "hmm", BTREE: "btree", HMM_CTX: "hmmctx"}
BASE_SEED = 2511113460


@dataclasses.dataclass(frozen=True)
class HeadShape:
    family: int
    n: int
    r: int
    v: int
    d: int
    io_dtype: int = BF16
    v_valid: int = 0          # symbols that exist when v is padded to a multiple of 16 (0: all v)

    @property
    def symbols(self) -> int:
        return self.v_valid or self.v

    @property
    def num_sum_groups(self) -> int:
        """Number of contextual sum units S (each has r weights produced from the hidden state)."""
        if self.family == BTREE:
            return 1 + (self.n - 2) * self.r
        if self.family == HMM_CTX:
            return 1 + (self.n - 1) * self.r
        return 1

    @property
    def sum_rows(self) -> int:
        return self.num_sum_groups * self.r


_CHUNK = 1 << 22


def _bf16_round_into(x: np.ndarray, out: np.ndarray) -> None:
    bits = x.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    out[...] = rounded.view(np.float32)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); returns fp32 holding bf16-representable values.
    Large arrays are processed in chunks on a thread pool (no array-sized temporaries)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    flat = x.reshape(-1)
    out = np.empty_like(flat)
    total = flat.size
    nchunks = (total + _CHUNK - 1) // _CHUNK
    if nchunks <= 1:
        _bf16_round_into(flat, out)
    else:
        def work(c):
            lo, hi = c * _CHUNK, min(total, (c + 1) * _CHUNK)
            _bf16_round_into(flat[lo:hi], out[lo:hi])
        with ThreadPoolExecutor(max_workers=8) as ex:
            list(ex.map(work, range(nchunks)))
    return out.reshape(x.shape)


def bf16_bits(x_rounded: np.ndarray) -> np.ndarray:
    """The uint16 bf16 bit patterns of values that are already bf16-representable."""
    x = np.ascontiguousarray(x_rounded, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def _normal(seed: int, stream: int, shape, std: float) -> np.ndarray:
    """N(0, std) fp32 tensor; chunk c of stream s comes from Philox(key=[seed, s * 2^20 + c]), so the
    values do not depend on how many threads fill the buffer."""
    total = int(np.prod(shape))
    out = np.empty(total, dtype=np.float32)
    nchunks = (total + _CHUNK - 1) // _CHUNK

    def fill(c):
        lo = c * _CHUNK
        hi = min(total, lo + _CHUNK)
        g = np.random.Generator(np.random.Philox(key=[seed, stream * (1 << 20) + c]))
        out[lo:hi] = g.standard_normal(hi - lo, dtype=np.float32) * np.float32(std)

    if nchunks == 1:
        fill(0)
    else:
        with ThreadPoolExecutor(max_workers=8) as ex:
            list(ex.map(fill, range(nchunks)))
    return out.reshape(shape)


def _gen(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, stream * (1 << 20)]))


def zipf_targets(seed: int, stream: int, shape, v: int, a: float = 1.1) -> np.ndarray:
    """Symbols whose RANKS follow a Zipf(a) law truncated to v; rank -> symbol by a seeded permutation."""
    g = _gen(seed, stream)
    pmf = 1.0 / np.arange(1, v + 1, dtype=np.float64) ** a
    pmf /= pmf.sum()
    ranks = g.choice(v, size=shape, p=pmf)
    perm = g.permutation(v)
    return perm[ranks].astype(np.int32)


def uniform_targets(seed: int, stream: int, shape, v: int) -> np.ndarray:
    return _gen(seed, stream).integers(0, v, size=shape, dtype=np.int32)


def uniforms(seed: int, stream: int, shape) -> np.ndarray:
    """fp32 uniforms in [0,1) on a 2^-24 grid (exactly representable, never 1.0)."""
    k = _gen(seed, stream).integers(0, 1 << 24, size=shape, dtype=np.int64)
    return (k.astype(np.float64) / float(1 << 24)).astype(np.float32)


def target_rows(seed: int, stream: int, shape, concentration: float = 0.3) -> np.ndarray:
    """Stand-in for a verifier LLM's next-byte distributions: fp32 rows on the simplex (last axis), drawn
    Dirichlet(concentration): peaked like byte-level LM predictions and unrelated to the draft head, so some
    drafted bytes get accepted and some rejected. No arithmetic of the method: gamma draws, normalised."""
    g = _gen(seed, stream).gamma(concentration, size=shape) + 1e-6
    return (g / g.sum(axis=-1, keepdims=True)).astype(np.float32)


@dataclasses.dataclass
class Workload:
    """Everything one call needs. `*_q` arrays are fp32 holding the bf16-rounded values both sides compute
    on; `hidden_raw` / `W_*_raw` are the un-rounded fp32 tensors, handed to the library only when io_dtype is F32."""
    name: str
    shape: HeadShape
    T: int
    hidden_q: np.ndarray
    W_emit_q: np.ndarray
    W_sum_q: np.ndarray
    T_static: np.ndarray | None
    targets: np.ndarray | None
    wpp: int = 0
    uniforms: np.ndarray | None = None
    hidden_raw: np.ndarray | None = None
    W_emit_raw: np.ndarray | None = None
    W_sum_raw: np.ndarray | None = None
    W_emit_dev_q: np.ndarray | None = None   # padded vocabulary: what the device gets ([n, r, v, d], padding rows filled
                                             # with noise); W_emit_q then holds the rows of the existing symbols only


_last_weights: dict = {}     # the most recent head's weights (one entry: they can be GBs)


def make_workload(name: str, shape: HeadShape, T: int, seed: int, *, target_kind: str | None = "uniform",
                  wpp: int = 0, weight_std: float = 0.02, trans_std: float = 1.0) -> Workload:
    hidden = _normal(seed, 1, (T, shape.d), 1.0)
    key = (seed, shape, weight_std, trans_std)
    if _last_weights.get("key") == key:          # cells that share a head (same seed and shape) reuse its weights
        W_emit, W_sum, T_static, W_emit_q, W_sum_q = _last_weights["value"]
    else:
        W_emit = _normal(seed, 2, (shape.n, shape.r, shape.v, shape.d), weight_std)
        W_sum = _normal(seed, 3, (shape.sum_rows, shape.d), weight_std)
        T_static = None
        if shape.family == HMM:
            T_static = _normal(seed, 4, (max(shape.n - 1, 1), shape.r, shape.r), trans_std)[: shape.n - 1]
        elif shape.family == HMM_CTX:
            # transition bias: a noisy multiple of the identity, as after training from the identity initialisation
            T_static = _normal(seed, 4, (max(shape.n - 1, 1), shape.r, shape.r), trans_std)[: shape.n - 1]
            T_static = T_static + np.float32(4.0) * np.eye(shape.r, dtype=np.float32)[None]
        W_emit_q, W_sum_q = bf16_round(W_emit), bf16_round(W_sum)
        if shape.io_dtype != F32:
            W_emit = W_sum = None                # only the rounded copies are kept
        _last_weights.clear()
        _last_weights.update(key=key, value=(W_emit, W_sum, T_static, W_emit_q, W_sum_q))
    targets = None
    if target_kind == "uniform":
        targets = uniform_targets(seed, 5, (T, shape.n), shape.symbols)
    elif target_kind == "zipf":
        targets = zipf_targets(seed, 5, (T, shape.n), shape.symbols)
    u = uniforms(seed, 6, (T * wpp, 2 * shape.n)) if wpp > 0 else None
    wl = Workload(name, shape, T, bf16_round(hidden), W_emit_q, W_sum_q, T_static, targets, wpp, u)
    if shape.io_dtype == F32:
        wl.hidden_raw, wl.W_emit_raw, wl.W_sum_raw = hidden, W_emit, W_sum
    if shape.v_valid:
        wl.W_emit_dev_q = W_emit_q
        wl.W_emit_q = np.ascontiguousarray(W_emit_q[:, :, :shape.v_valid, :])
    return wl


def lowrank_parameters(n: int, r: int, v: int, d: int, k: int, seed: int, *, weight_std: float = 0.02,
                       adaptor_std: float = 0.05, zero_B: bool = False):
    """Seeded parameters of the shared-unembedding parametrisation (App. G): W_base [n, v, d], A [n, r, v, k],
    B [n, r, k, d] as fp32 arrays of bf16-representable values. zero_B gives the initialisation App. G proposes
    (every adaptor starts at zero)."""
    W_base = bf16_round(_normal(seed, 11, (n, v, d), weight_std))
    A = bf16_round(_normal(seed, 12, (n, r, v, k), adaptor_std))
    B = np.zeros((n, r, k, d), dtype=np.float32) if zero_B else bf16_round(_normal(seed, 13, (n, r, k, d), adaptor_std))
    return W_base, A, B


def lowrank_upstream_gradient(n: int, r: int, v: int, d: int, seed: int) -> np.ndarray:
    """A seeded stand-in for the gradient of the composed unembeddings, [n, r, v, d] fp32."""
    return _normal(seed, 14, (n, r, v, d), 1.0)


DECODE_CELLS = [(fam, n, P) for fam in (CP, HMM) for n in (8, 16) for P in (1, 8, 64)]


def config_workload(idx: int, *, cell: tuple[int, int, int] | None = None, T: int | None = None) -> Workload:
    """The five named workloads. `T` overrides the number of positions (used for scaled-down captures);
    for idx 4 `cell` = (family, n, P) picks one cell of the decode sweep."""
    seed = BASE_SEED + idx
    if idx == 0:
        return make_workload("cp_tiny", HeadShape(CP, 4, 8, 256, 256, F32), T or 256, seed,
                             target_kind="uniform", wpp=1)
    if idx == 1:
        return make_workload("cp_train", HeadShape(CP, 8, 16, 320, 4096), T or 8192, seed, target_kind="zipf")
    if idx == 2:
        return make_workload("hmm_train", HeadShape(HMM, 8, 32, 320, 4096), T or 8192, seed, target_kind="zipf")
    if idx == 3:
        return make_workload("btree_train", HeadShape(BTREE, 16, 32, 256, 3072), T or 4096, seed,
                             target_kind="uniform", wpp=1)
    if idx == 6:
        return make_workload("cp_llama_byte", HeadShape(CP, 8, 16, 272, 3072, F32, v_valid=268), T or 8192, seed,
                             target_kind="zipf")      # fp32 tensors in, as the paper runs its byte-level Llama (Table 4)
    if idx == 5:
        return make_workload("hmmctx_train", HeadShape(HMM_CTX, 8, 32, 320, 4096), T or 8192, seed, target_kind="zipf")
    if idx == 4:
        fam, n, P = cell or (CP, 8, 8)
        r = 16 if fam == CP else 32          # HMM and HMM_CTX
        cseed = seed + 1000 * (fam * 2 + (n // 8 - 1))   # weights shared by the three P of a (family, n)
        return make_workload(f"decode_{FAMILY_NAMES[fam]}_n{n}_P{P}", HeadShape(fam, n, r, 320, 4096), T or P,
                             cseed, target_kind=None, wpp=16)
    raise ValueError(f"no such config {idx}")
