"""Seeded synthetic workloads for shared-prefix decode attention.

This module only draws numbers and lays them out in pages.  It holds none of
the attention arithmetic: no scores, no softmax, no merge.  Both the CPU
oracle's tests and the CUDA path's tests/bench take their inputs from here.

Workload shape (why it looks like this): the max-reward search of Section 2.2
samples k candidate programs from ONE state s_i, so all k rollouts of a round
share the whole prompt; Section 3.1 ("Experimental Setup") fixes K = 8
candidates x depth 8 and the flat-sampling baseline draws n = 64 completions
of a single prompt; prompts carry the whole trajectory and its critiques
(Section 3.2, RQ2), so the shared prefix is thousands of tokens long, and
critiques are produced with extended thinking, so some rollouts are very long.
The five configurations below encode those shapes as G prompt groups x C
candidates, one shared prefix per group and one private suffix per candidate.

Storage layout produced here (and consumed by the CUDA library):
  K pool, V pool : [num_pages][Hkv][page][d] one (page, kv-head) slab is
                                              page*d contiguous elements (page = 16
                                              tokens unless the configuration says 32 or 64)
  prefix_pages   : int32 [G][max_prefix_pages]
  suffix_pages   : int32 [B][max_suffix_pages]
  prefix_len     : int32 [G]      tokens
  suffix_len     : int32 [B]      tokens
  group_offsets  : int32 [G+1]    candidates of a group are contiguous in b

bf16 tensors are carried on the host as uint16 bit patterns (numpy has no
bf16); `bf16_bits_to_f32` widens them exactly.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

PAGE = 16

# tensor ids for sub-stream derivation: (seed, tensor id, index) -> SeedSequence
_T_PREFIX_LEN, _T_SUFFIX_LEN, _T_PERM, _T_Q, _T_KP, _T_VP, _T_KS, _T_VS, _T_OUTLIER, _T_KNEW, _T_VNEW = range(11)
_T_HIDDEN, _T_WQKV, _T_BQKV = 11, 12, 13

# Finite, large filler for page slots past a sequence's length: a kernel that
# fails to mask them produces visibly wrong results instead of silently
# averaging plausible numbers.
SENTINEL = 1.0e4


def _rng(seed: int, tensor: int, index: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([seed, tensor, index])))


# ----------------------------------------------------------------------------
# bf16 <-> f32 bit conversions (round-to-nearest-even), numpy only
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even.  Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> float32, exact."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# configurations
# ----------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    dtype: str                      # "f32" | "bf16" | "fp8" (e4m3 cache with per-page scales; q, o, new tokens bf16)
    G: int                          # prompt groups
    C: int                          # candidates per group
    Hq: int
    Hkv: int
    d: int
    prefix: Tuple                   # ("fixed", P) | ("loguniform", lo, hi)
    suffix: Tuple                   # ("fixed", (s0, s1, ...)) | ("uniform", lo, hi)
    permute_pages: bool = False
    k_outlier_prob: float = 0.0     # probability that a K token row is an outlier
    k_outlier_scale: float = 1.0
    append_steps: int = 0           # extra decode steps, one appended token per candidate each
    seed: int = 0
    page: int = PAGE                # tokens per cache page: 16, 32 or 64

    @property
    def B(self) -> int:
        return self.G * self.C

    @property
    def g(self) -> int:
        return self.Hq // self.Hkv

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    @property
    def elem_bytes(self) -> int:
        """Bytes per element of q, o and the appended rows."""
        return 4 if self.dtype == "f32" else 2

    @property
    def kv_elem_bytes(self) -> int:
        """Bytes per cached K or V element."""
        return 1 if self.dtype == "fp8" else self.elem_bytes


CONFIGS: Dict[str, Config] = {
    # tiny fp32 case: one group of 4 candidates, fixed suffix lengths
    "cfg0": Config("cfg0", "f32", 1, 4, 4, 1, 64, ("fixed", 256), ("fixed", (0, 17, 40, 64))),
    # one round of K=8 candidates from one state
    "cfg1": Config("cfg1", "bf16", 1, 8, 32, 8, 128, ("fixed", 2048), ("uniform", 0, 1024), permute_pages=True),
    # flat sampling, n=64 completions of one prompt, 32 consecutive decode steps
    "cfg2": Config("cfg2", "bf16", 1, 64, 64, 8, 128, ("fixed", 8192), ("uniform", 0, 4096),
                   permute_pages=True, append_steps=32),
    # 16 problems x 16 candidates, ragged prompts, K outliers
    "cfg3": Config("cfg3", "bf16", 16, 16, 32, 8, 128, ("loguniform", 1024, 16384), ("uniform", 0, 8192),
                   k_outlier_prob=0.01, k_outlier_scale=8.0),
    # long-reasoning rollouts (extended-thinking critiques)
    "cfg4": Config("cfg4", "bf16", 4, 32, 64, 8, 128, ("fixed", 4096), ("uniform", 16384, 32768),
                   permute_pages=True, append_steps=64),
    # cfg4 over an e4m3 cache with per-(page, kv head) scales: half the bytes per cached token
    "cfg4_fp8": Config("cfg4_fp8", "fp8", 4, 32, 64, 8, 128, ("fixed", 4096), ("uniform", 16384, 32768),
                       permute_pages=True, append_steps=64),
    # eight of cfg3's sixteen problems (2.3 GB): the same chunk geometry and one-row-tile prefix items at a size a
    # profiler can replay
    "cfg3g8": Config("cfg3g8", "bf16", 8, 16, 32, 8, 128, ("loguniform", 1024, 16384), ("uniform", 0, 8192),
                     k_outlier_prob=0.01, k_outlier_scale=8.0),
    # one of cfg4's four prompt groups alone (3.2 GB): the same chunk geometry at a size a profiler can replay
    "cfg4g1": Config("cfg4g1", "bf16", 1, 32, 64, 8, 128, ("fixed", 4096), ("uniform", 16384, 32768),
                     permute_pages=True, append_steps=64),
}


def scaled_down(cfg: Config, name: str, *, G=None, C=None, prefix=None, suffix=None, append_steps=None,
                permute_pages=None) -> Config:
    """A smaller instance with the same structure, for cases the CPU oracle checks in full."""
    kw = {}
    for k, v in dict(G=G, C=C, prefix=prefix, suffix=suffix, append_steps=append_steps,
                     permute_pages=permute_pages).items():
        if v is not None:
            kw[k] = v
    return dataclasses.replace(cfg, name=name, **kw)


# ----------------------------------------------------------------------------
# lengths and page tables
# ----------------------------------------------------------------------------
def draw_lengths(cfg: Config) -> Tuple[np.ndarray, np.ndarray]:
    """prefix_len[G], suffix_len[B] (int32).  Uniform: integers, both ends inclusive, i.i.d.
    Log-uniform: round(exp(U(ln lo, ln hi))) clamped to [lo, hi], i.i.d. per group."""
    kind = cfg.prefix[0]
    if kind == "fixed":
        prefix_len = np.full(cfg.G, cfg.prefix[1], dtype=np.int32)
    elif kind == "loguniform":
        lo, hi = cfg.prefix[1], cfg.prefix[2]
        u = _rng(cfg.seed, _T_PREFIX_LEN).uniform(math.log(lo), math.log(hi), size=cfg.G)
        prefix_len = np.clip(np.rint(np.exp(u)), lo, hi).astype(np.int32)
    else:
        raise ValueError(kind)
    kind = cfg.suffix[0]
    if kind == "fixed":
        vals = np.asarray(cfg.suffix[1], dtype=np.int32)
        suffix_len = np.resize(vals, cfg.B).astype(np.int32)
    elif kind == "uniform":
        lo, hi = cfg.suffix[1], cfg.suffix[2]
        suffix_len = _rng(cfg.seed, _T_SUFFIX_LEN).integers(lo, hi + 1, size=cfg.B).astype(np.int32)
    else:
        raise ValueError(kind)
    return prefix_len, suffix_len


@dataclasses.dataclass
class PageTables:
    num_pages: int
    max_prefix_pages: int
    max_suffix_pages: int
    prefix_pages: np.ndarray        # int32 [G][max_prefix_pages], unused entries -1
    suffix_pages: np.ndarray        # int32 [B][max_suffix_pages], unused entries -1
    group_offsets: np.ndarray       # int32 [G+1]


def build_page_tables(cfg: Config, prefix_len: np.ndarray, suffix_len: np.ndarray,
                      headroom_tokens: Optional[int] = None, permute: Optional[bool] = None) -> PageTables:
    """Assign physical pages.  A prefix occupies ceil(P/page) pages (the last one possibly partial); every
    candidate's suffix starts on a fresh page of its own and is pre-assigned enough pages for
    `headroom_tokens` appended tokens, so appends never need an allocator.  With `permute`, one uniform
    random permutation over all physical page ids of the pool is applied (Fisher-Yates, seeded)."""
    if headroom_tokens is None:
        headroom_tokens = cfg.append_steps + 1
    if permute is None:
        permute = cfg.permute_pages
    npp = (prefix_len.astype(np.int64) + cfg.page - 1) // cfg.page
    nsp = (suffix_len.astype(np.int64) + headroom_tokens + cfg.page - 1) // cfg.page
    num_pages = int(npp.sum() + nsp.sum())
    max_pp = max(1, int(npp.max(initial=0)))
    max_sp = max(1, int(nsp.max(initial=0)))
    ids = np.arange(num_pages, dtype=np.int32)
    if permute:
        ids = _rng(cfg.seed, _T_PERM).permutation(num_pages).astype(np.int32)
    prefix_pages = np.full((cfg.G, max_pp), -1, dtype=np.int32)
    suffix_pages = np.full((cfg.B, max_sp), -1, dtype=np.int32)
    cur = 0
    for j in range(cfg.G):
        n = int(npp[j])
        prefix_pages[j, :n] = ids[cur:cur + n]
        cur += n
    for b in range(cfg.B):
        n = int(nsp[b])
        suffix_pages[b, :n] = ids[cur:cur + n]
        cur += n
    assert cur == num_pages
    group_offsets = (np.arange(cfg.G + 1, dtype=np.int64) * cfg.C).astype(np.int32)
    return PageTables(num_pages, max_pp, max_sp, prefix_pages, suffix_pages, group_offsets)


# ----------------------------------------------------------------------------
# values
# ----------------------------------------------------------------------------
def _normal(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(size=shape, dtype=np.float32)


def _round_to_dtype(cfg: Config, x: np.ndarray) -> np.ndarray:
    """Round float32 draws to the storage dtype; returns float32 holding exactly representable values."""
    if cfg.dtype == "f32":
        return x
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


def storage_array(cfg: Config, x: np.ndarray) -> np.ndarray:
    """float32 values (already representable) -> storage array: float32, or uint16 bf16 bits."""
    if cfg.dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    return f32_to_bf16_bits(x)


def _draw_k(cfg: Config, tensor: int, index: int, n_tokens: int) -> np.ndarray:
    """K rows [n_tokens][Hkv][d]; with probability k_outlier_prob a whole token row (per kv head) is
    multiplied by k_outlier_scale before rounding."""
    k = _normal(_rng(cfg.seed, tensor, index), (n_tokens, cfg.Hkv, cfg.d))
    if cfg.k_outlier_prob > 0.0:
        mask = _rng(cfg.seed, _T_OUTLIER, index * 2 + (0 if tensor == _T_KP else 1)).random((n_tokens, cfg.Hkv)) \
            < cfg.k_outlier_prob
        k = np.where(mask[:, :, None], k * np.float32(cfg.k_outlier_scale), k)
    return _round_to_dtype(cfg, k)


def draw_q(cfg: Config, step: int = 0) -> np.ndarray:
    """Queries [B][Hq][d] for decode step `step`, float32 holding storage-representable values."""
    return _round_to_dtype(cfg, _normal(_rng(cfg.seed, _T_Q, step), (cfg.B, cfg.Hq, cfg.d)))


def draw_append(cfg: Config, step: int) -> Tuple[np.ndarray, np.ndarray]:
    """New token's K and V, [B][Hkv][d] each, appended before decode step `step` (step >= 1)."""
    k = _round_to_dtype(cfg, _normal(_rng(cfg.seed, _T_KNEW, step), (cfg.B, cfg.Hkv, cfg.d)))
    v = _round_to_dtype(cfg, _normal(_rng(cfg.seed, _T_VNEW, step), (cfg.B, cfg.Hkv, cfg.d)))
    return k, v


def draw_hidden(cfg: Config, step: int, hidden: int) -> np.ndarray:
    """Hidden states [B][hidden] entering the projection of decode step `step`: N(0, 1), bf16-representable float32."""
    return bf16_bits_to_f32(f32_to_bf16_bits(_normal(_rng(cfg.seed, _T_HIDDEN, step), (cfg.B, hidden))))


def draw_qkv_weights(cfg: Config, hidden: int, with_bias: bool = True) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    """Projection weights [(Hq + 2 Hkv) d][hidden], N(0, 1 / hidden) so that a projected feature is N(0, 1) like the
    queries and keys of the other generators, and a bias [(Hq + 2 Hkv) d], N(0, 0.25); bf16-representable float32."""
    n = (cfg.Hq + 2 * cfg.Hkv) * cfg.d
    w = _normal(_rng(cfg.seed, _T_WQKV), (n, hidden)) * np.float32(1.0 / math.sqrt(hidden))
    b = _normal(_rng(cfg.seed, _T_BQKV), (n,)) * np.float32(0.5) if with_bias else None
    rnd = lambda a: bf16_bits_to_f32(f32_to_bf16_bits(np.ascontiguousarray(a, dtype=np.float32)))
    return rnd(w), (rnd(b) if b is not None else None)


def draw_single_head_history(cfg: Config, index: int, n_tokens: int) -> Tuple[np.ndarray, np.ndarray]:
    """K [n][d] and V [n][d] of ONE kv head with the configuration's value distribution (outlier rows
    included), for timing or checking a single (candidate, head) row without building whole pools."""
    k = _normal(_rng(cfg.seed, _T_KS, 1_000_000 + index), (n_tokens, cfg.d))
    if cfg.k_outlier_prob > 0.0:
        mask = _rng(cfg.seed, _T_OUTLIER, 1_000_000 + index).random(n_tokens) < cfg.k_outlier_prob
        k = np.where(mask[:, None], k * np.float32(cfg.k_outlier_scale), k)
    v = _normal(_rng(cfg.seed, _T_VS, 1_000_000 + index), (n_tokens, cfg.d))
    return _round_to_dtype(cfg, k), _round_to_dtype(cfg, v)


@dataclasses.dataclass
class HostProblem:
    """A fully host-resident instance: the logical (unpaged) K/V and, built from it by a separate
    scatter, the paged pool image."""
    cfg: Config
    prefix_len: np.ndarray
    suffix_len: np.ndarray          # current lengths (grow with append())
    tables: PageTables
    k_prefix: List[np.ndarray]      # per group  [P_j][Hkv][d] float32
    v_prefix: List[np.ndarray]
    k_suffix: List[np.ndarray]      # per candidate [s_b][Hkv][d] float32 (grows with append())
    v_suffix: List[np.ndarray]
    k_pool: np.ndarray              # [num_pages][Hkv][page][d] storage dtype
    v_pool: np.ndarray
    outer: List["HostLevel"] = dataclasses.field(default_factory=list)   # outer cascade levels, if any

    def group_of(self, b: int) -> int:
        return int(np.searchsorted(self.tables.group_offsets, b, side="right") - 1)

    def append(self, k_new: np.ndarray, v_new: np.ndarray) -> None:
        """Host mirror of one append step: extends the logical suffixes (the pool image is not touched;
        the device pool is updated by the library's own append)."""
        for b in range(self.cfg.B):
            self.k_suffix[b] = np.concatenate([self.k_suffix[b], k_new[b][None]], axis=0)
            self.v_suffix[b] = np.concatenate([self.v_suffix[b], v_new[b][None]], axis=0)
        self.suffix_len = self.suffix_len + 1


@dataclasses.dataclass
class HostLevel:
    """One outer level of a prefix cascade: token ranges shared by more candidates than the base groups."""
    group_offsets: np.ndarray       # int32 [n_groups+1], candidates contiguous in b
    length: np.ndarray              # int32 [n_groups]
    pages: np.ndarray               # int32 [n_groups][max_pages]
    k: List[np.ndarray]             # per outer group [len][Hkv][d] float32
    v: List[np.ndarray]


def add_outer_level(hp: "HostProblem", group_offsets: Sequence[int], lengths: Sequence[int], level_index: int = 0
                    ) -> HostLevel:
    """Appends an outer cascade level to a host problem: draws its K/V, gives it fresh pages at the end of the
    pools (permuted among themselves when the configuration permutes pages) and scatters them in."""
    cfg = hp.cfg
    lengths = np.asarray(lengths, dtype=np.int32)
    go = np.asarray(group_offsets, dtype=np.int32)
    n_groups = len(lengths)
    npp = (lengths.astype(np.int64) + cfg.page - 1) // cfg.page
    first = hp.k_pool.shape[0]
    extra = int(npp.sum())
    ids = np.arange(first, first + extra, dtype=np.int32)
    if cfg.permute_pages:
        ids = ids[_rng(cfg.seed, _T_PERM, 100 + level_index).permutation(extra)]
    fill = storage_array(cfg, np.full(1, SENTINEL, dtype=np.float32))[0]
    pad = np.full((extra,) + hp.k_pool.shape[1:], fill, dtype=hp.k_pool.dtype)
    hp.k_pool = np.concatenate([hp.k_pool, pad], axis=0)
    hp.v_pool = np.concatenate([hp.v_pool, pad.copy()], axis=0)
    hp.tables.num_pages = first + extra
    max_pages = max(1, int(npp.max(initial=0)))
    pages = np.full((n_groups, max_pages), -1, dtype=np.int32)
    ks, vs, cur = [], [], 0
    for j in range(n_groups):
        n = int(npp[j])
        pages[j, :n] = ids[cur:cur + n]
        cur += n
        ks.append(_draw_k(cfg, _T_KP, 1000 * (level_index + 1) + j, int(lengths[j])))
        vs.append(_round_to_dtype(cfg, _normal(_rng(cfg.seed, _T_VP, 1000 * (level_index + 1) + j),
                                               (int(lengths[j]), cfg.Hkv, cfg.d))))
        _scatter(hp.k_pool, pages[j], ks[j], cfg)
        _scatter(hp.v_pool, pages[j], vs[j], cfg)
    lvl = HostLevel(go, lengths, pages, ks, vs)
    hp.outer.append(lvl)
    return lvl


def _scatter(pool: np.ndarray, pages_row: np.ndarray, tokens: np.ndarray, cfg: Config) -> None:
    """Write logical rows tokens[n][Hkv][d] into the pool through one page-table row."""
    n = tokens.shape[0]
    st = storage_array(cfg, tokens)
    page = pool.shape[2]
    for p in range((n + page - 1) // page):
        lo, hi = p * page, min(n, (p + 1) * page)
        pid = int(pages_row[p])
        # pool[pid] is [Hkv][page][d]; tokens are [t][Hkv][d]
        pool[pid, :, :hi - lo, :] = np.transpose(st[lo:hi], (1, 0, 2))


def make_host_problem(cfg: Config, *, headroom_tokens: Optional[int] = None, permute: Optional[bool] = None,
                      prefix_len: Optional[np.ndarray] = None, suffix_len: Optional[np.ndarray] = None
                      ) -> HostProblem:
    if prefix_len is None or suffix_len is None:
        pl, sl = draw_lengths(cfg)
        prefix_len = pl if prefix_len is None else np.asarray(prefix_len, dtype=np.int32)
        suffix_len = sl if suffix_len is None else np.asarray(suffix_len, dtype=np.int32)
    tables = build_page_tables(cfg, prefix_len, suffix_len, headroom_tokens, permute)
    k_prefix = [_draw_k(cfg, _T_KP, j, int(prefix_len[j])) for j in range(cfg.G)]
    v_prefix = [_round_to_dtype(cfg, _normal(_rng(cfg.seed, _T_VP, j), (int(prefix_len[j]), cfg.Hkv, cfg.d)))
                for j in range(cfg.G)]
    k_suffix = [_draw_k(cfg, _T_KS, b, int(suffix_len[b])) for b in range(cfg.B)]
    v_suffix = [_round_to_dtype(cfg, _normal(_rng(cfg.seed, _T_VS, b), (int(suffix_len[b]), cfg.Hkv, cfg.d)))
                for b in range(cfg.B)]
    shape = (tables.num_pages, cfg.Hkv, cfg.page, cfg.d)
    fill = storage_array(cfg, np.full(1, SENTINEL, dtype=np.float32))[0]
    k_pool = np.full(shape, fill, dtype=fill.dtype)
    v_pool = np.full(shape, fill, dtype=fill.dtype)
    for j in range(cfg.G):
        _scatter(k_pool, tables.prefix_pages[j], k_prefix[j], cfg)
        _scatter(v_pool, tables.prefix_pages[j], v_prefix[j], cfg)
    for b in range(cfg.B):
        _scatter(k_pool, tables.suffix_pages[b], k_suffix[b], cfg)
        _scatter(v_pool, tables.suffix_pages[b], v_suffix[b], cfg)
    return HostProblem(cfg, prefix_len.copy(), suffix_len.copy(), tables, k_prefix, v_prefix, k_suffix, v_suffix,
                       k_pool, v_pool)


# ----------------------------------------------------------------------------
# accounting (bytes that any implementation must move at least once)
# ----------------------------------------------------------------------------
def unique_bytes(cfg: Config, prefix_len: np.ndarray, suffix_len: np.ndarray) -> Dict[str, int]:
    """Minimum unique traffic of one decode step: every valid prefix token once per group, every valid
    suffix token once, all KV heads, K and V; plus Q read, O write, LSE write."""
    per_tok = 2 * cfg.Hkv * cfg.d * cfg.kv_elem_bytes
    kv_prefix = int(prefix_len.astype(np.int64).sum()) * per_tok
    kv_suffix = int(suffix_len.astype(np.int64).sum()) * per_tok
    if cfg.dtype == "fp8":           # plus the K and the V scale of every page that holds a token, per kv head
        pages = lambda n: int(((n.astype(np.int64) + PAGE - 1) // PAGE).sum())
        kv_prefix += pages(prefix_len) * 2 * cfg.Hkv * 4
        kv_suffix += pages(suffix_len) * 2 * cfg.Hkv * 4
    qo = 2 * cfg.B * cfg.Hq * cfg.d * cfg.elem_bytes
    lse = cfg.B * cfg.Hq * 4
    return {"kv_prefix": kv_prefix, "kv_suffix": kv_suffix, "q_o": qo, "lse": lse,
            "total": kv_prefix + kv_suffix + qo + lse}


def gather_logical(pool: np.ndarray, pages_row: Sequence[int], n_tokens: int, h: int) -> np.ndarray:
    """Read n_tokens rows of kv head h back out of a pool image through a page-table row:
    returns [n_tokens][d] in the pool's storage dtype.  Plain indexing, used by tests that hold only the
    paged image (device-generated pools)."""
    page = pool.shape[2]
    n_pages = (n_tokens + page - 1) // page
    if n_pages == 0:
        return np.zeros((0, pool.shape[-1]), dtype=pool.dtype)
    ids = np.asarray(pages_row[:n_pages], dtype=np.int64)
    return pool[ids, h].reshape(n_pages * page, pool.shape[-1])[:n_tokens]


# ----------------------------------------------------------------------------
# search bookkeeping: a batch of trajectories
# ----------------------------------------------------------------------------
SEARCH_THRESHOLDS = (120.0, 200.0, 300.0)      # s1, s2, s3 in percent (the paper leaves them open)


def draw_search_batch(problems: int, K: int = 8, T: int = 8, seed: int = 0, ragged: bool = True):
    """`problems` optimisation problems with K trajectories of at most T steps each (Section 3.1: K = 8, depth 8).
    Returns a dict of step-major float32 / uint8 / int32 arrays: speed-ups in percent (log-normal around 100,
    heavy right tail like measured kernel speed-ups), correctness (70 % pass), lengths (uniform 1..T when ragged),
    value-head logits N(0, 2) for the last state of every trajectory, and the group offsets of the problems."""
    N = problems * K
    rng = np.random.Generator(np.random.Philox(np.random.SeedSequence([seed, 77, N, T])))
    speedup = (100.0 * np.exp(rng.normal(0.1, 0.6, size=(T, N)))).astype(np.float32)
    correct = (rng.random((T, N)) < 0.7).astype(np.uint8)
    length = rng.integers(1, T + 1, size=N).astype(np.int32) if ragged else np.full(N, T, dtype=np.int32)
    logits = rng.normal(0.0, 2.0, size=(N, 5)).astype(np.float32)
    group_offsets = (np.arange(problems + 1) * K).astype(np.int32)
    return {"speedup": speedup, "correct": correct, "len": length, "logits": logits, "group_offsets": group_offsets,
            "N": N, "T": T, "P": problems}


# ----------------------------------------------------------------------------
# scoring: whole sequences behind a shared prompt, one query per token
# ----------------------------------------------------------------------------
@dataclasses.dataclass
class ScoringHostProblem:
    """G prompt groups x C sequences; every token of every sequence is a query (a "virtual candidate", numbered
    sequence by sequence, position by position).  Logical K/V plus the paged pool image and the tables that describe
    it to the library as a cascade: base level = the prompts, one outer level = each sequence's own tokens."""
    cfg: Config                       # dtype / heads / d; G, C as given
    prefix_len: np.ndarray            # int32 [G]
    seq_len: np.ndarray               # int32 [G*C]
    k_prefix: List[np.ndarray]
    v_prefix: List[np.ndarray]
    k_seq: List[np.ndarray]           # per sequence [n_b][Hkv][d] float32
    v_seq: List[np.ndarray]
    k_pool: np.ndarray
    v_pool: np.ndarray
    prefix_pages: np.ndarray          # int32 [G][max_prefix_pages]
    seq_pages: np.ndarray             # int32 [G*C][max_seq_pages]
    group_offsets: np.ndarray         # int32 [G+1] over virtual candidates (base level)
    seq_offsets: np.ndarray           # int32 [G*C+1] over virtual candidates (outer level)
    row_limit: np.ndarray             # int32 [B']: position + 1


def make_scoring_host_problem(cfg: Config, prefix_len: Sequence[int], seq_len: Sequence[int],
                              last_queries: Optional[int] = None) -> ScoringHostProblem:
    """`last_queries` = None: every token of a sequence is a query (scoring).  `last_queries` = n: only the last n
    tokens of every sequence are queries (a decode step that verifies n speculated tokens at once); the virtual
    candidates of sequence b are then its positions max(0, n_b - n) .. n_b - 1."""
    prefix_len = np.asarray(prefix_len, dtype=np.int32)
    seq_len = np.asarray(seq_len, dtype=np.int32)
    assert len(prefix_len) == cfg.G and len(seq_len) == cfg.B
    npp = (prefix_len.astype(np.int64) + PAGE - 1) // PAGE
    nsp = (seq_len.astype(np.int64) + PAGE - 1) // PAGE
    num_pages = int(npp.sum() + nsp.sum()) + 1                        # one spare page so that the pool is never empty
    ids = np.arange(num_pages, dtype=np.int32)
    if cfg.permute_pages:
        ids = ids[_rng(cfg.seed, _T_PERM, 500).permutation(num_pages)]
    prefix_pages = np.full((cfg.G, max(1, int(npp.max(initial=0)))), -1, dtype=np.int32)
    seq_pages = np.full((cfg.B, max(1, int(nsp.max(initial=0)))), -1, dtype=np.int32)
    cur = 0
    for j in range(cfg.G):
        prefix_pages[j, :int(npp[j])] = ids[cur:cur + int(npp[j])]
        cur += int(npp[j])
    for b in range(cfg.B):
        seq_pages[b, :int(nsp[b])] = ids[cur:cur + int(nsp[b])]
        cur += int(nsp[b])
    k_prefix = [_draw_k(cfg, _T_KP, 5000 + j, int(prefix_len[j])) for j in range(cfg.G)]
    v_prefix = [_round_to_dtype(cfg, _normal(_rng(cfg.seed, _T_VP, 5000 + j), (int(prefix_len[j]), cfg.Hkv, cfg.d)))
                for j in range(cfg.G)]
    k_seq = [_draw_k(cfg, _T_KS, 5000 + b, int(seq_len[b])) for b in range(cfg.B)]
    v_seq = [_round_to_dtype(cfg, _normal(_rng(cfg.seed, _T_VS, 5000 + b), (int(seq_len[b]), cfg.Hkv, cfg.d)))
             for b in range(cfg.B)]
    shape = (num_pages, cfg.Hkv, PAGE, cfg.d)
    fill = storage_array(cfg, np.full(1, SENTINEL, dtype=np.float32))[0]
    k_pool = np.full(shape, fill, dtype=fill.dtype)
    v_pool = np.full(shape, fill, dtype=fill.dtype)
    for j in range(cfg.G):
        _scatter(k_pool, prefix_pages[j], k_prefix[j], cfg)
        _scatter(v_pool, prefix_pages[j], v_prefix[j], cfg)
    for b in range(cfg.B):
        _scatter(k_pool, seq_pages[b], k_seq[b], cfg)
        _scatter(v_pool, seq_pages[b], v_seq[b], cfg)
    n_query = seq_len if last_queries is None else np.minimum(seq_len, last_queries)
    seq_offsets = np.concatenate([[0], np.cumsum(n_query)]).astype(np.int32)
    group_offsets = seq_offsets[::cfg.C].copy()
    row_limit = np.concatenate([np.arange(n - nq + 1, n + 1) for n, nq in zip(seq_len, n_query)] +
                               [np.zeros(0)]).astype(np.int32)
    return ScoringHostProblem(cfg, prefix_len, seq_len, k_prefix, v_prefix, k_seq, v_seq, k_pool, v_pool, prefix_pages,
                              seq_pages, group_offsets, seq_offsets, row_limit)


def draw_scoring_q(cfg: Config, seq_len: Sequence[int], step: int = 0) -> List[np.ndarray]:
    """One query per token of every sequence: list of [n_b][Hq][d] float32 (storage-representable).  (When only the
    last n tokens are queries, take the last n rows of each.)"""
    return [_round_to_dtype(cfg, _normal(_rng(cfg.seed, _T_Q, 9000 + 100 * step + b), (int(n), cfg.Hq, cfg.d)))
            for b, n in enumerate(seq_len)]
