"""Device-side set-up shared by tests, the smoke check and the benchmark: moves a workload to the GPU as
torch tensors and wraps the layout handle.  Memory and marshalling only; all arithmetic happens in the
library's kernels."""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import binding as mc
from . import workload as wl


def to_device(cfg: wl.Config, x: np.ndarray, device="cuda") -> torch.Tensor:
    """float32 values (storage-representable) -> device tensor of the storage dtype."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    if cfg.dtype != "f32":
        t = t.to(torch.bfloat16)
    return t.to(device)


def storage_to_device(cfg: wl.Config, a: np.ndarray, device="cuda") -> torch.Tensor:
    """Storage array (float32, uint16 bf16 bits, or uint8 e4m3 codes) -> device tensor."""
    if cfg.dtype == "f32" or a.dtype == np.uint8:
        return torch.from_numpy(a).to(device)
    return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)


class DeviceProblem:
    """Pools, tables and lengths on the device plus the library's layout handle and workspace."""

    def __init__(self, cfg: wl.Config, tables: wl.PageTables, prefix_len: np.ndarray, suffix_len: np.ndarray,
                 k_pool: torch.Tensor, v_pool: torch.Tensor, device="cuda", outer=(), k_scale=None, v_scale=None):
        """k_scale, v_scale: float32 [num_pages][Hkv] device tensors, for an e4m3 cache (cfg.dtype == "fp8")."""
        self.cfg, self.tables, self.device = cfg, tables, device
        self.k_pool, self.v_pool = k_pool, v_pool
        self.k_scale, self.v_scale = k_scale, v_scale
        i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
        self.prefix_pages, self.suffix_pages = i32(tables.prefix_pages), i32(tables.suffix_pages)
        self.prefix_len, self.suffix_len = i32(prefix_len), i32(suffix_len)
        self.group_offsets = i32(tables.group_offsets)
        d = mc.LayoutDesc()
        d.num_groups, d.batch, d.num_q_heads, d.num_kv_heads, d.head_dim = cfg.G, cfg.B, cfg.Hq, cfg.Hkv, cfg.d
        d.page_size, d.num_pages = cfg.page, tables.num_pages
        d.max_prefix_pages, d.max_suffix_pages = tables.max_prefix_pages, tables.max_suffix_pages
        d.dtype = {"f32": mc.MC_F32, "bf16": mc.MC_BF16, "fp8": mc.MC_FP8_E4M3}[cfg.dtype]
        d.k_pool, d.v_pool = k_pool.data_ptr(), v_pool.data_ptr()
        if cfg.dtype == "fp8":
            d.k_scale, d.v_scale = k_scale.data_ptr(), v_scale.data_ptr()
        d.group_offsets, d.prefix_pages = self.group_offsets.data_ptr(), self.prefix_pages.data_ptr()
        d.prefix_len, d.suffix_pages = self.prefix_len.data_ptr(), self.suffix_pages.data_ptr()
        d.suffix_len = self.suffix_len.data_ptr()
        self.desc = d
        # outer cascade levels: (group_offsets, lengths, pages) numpy triples
        self.outer_tensors, levels = [], []
        for (go, ln, pg) in outer:
            t = (i32(go), i32(ln), i32(pg))
            self.outer_tensors.append(t)
            lv = mc.PrefixLevel()
            lv.num_groups, lv.max_pages = len(ln), pg.shape[1]
            lv.group_offsets, lv.len, lv.pages = t[0].data_ptr(), t[1].data_ptr(), t[2].data_ptr()
            levels.append(lv)
        self.layout = mc.mc_kv_layout_create_cascade(d, levels) if levels else mc.mc_kv_layout_create(d)
        self.geom = mc.mc_kv_layout_geometry(self.layout)
        self.ws_bytes = mc.mc_workspace_bytes(self.layout)
        self.ws = torch.empty(self.ws_bytes + 256, dtype=torch.uint8, device=device)
        self.ws_ptr = (self.ws.data_ptr() + 255) // 256 * 256
        self.tdtype = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
        self.o = torch.empty(cfg.B, cfg.Hq, cfg.d, dtype=self.tdtype, device=device)
        self.lse = torch.empty(cfg.B, cfg.Hq, dtype=torch.float32, device=device)

    @classmethod
    def from_host(cls, hp: wl.HostProblem, device="cuda") -> "DeviceProblem":
        return cls(hp.cfg, hp.tables, hp.prefix_len, hp.suffix_len,
                   storage_to_device(hp.cfg, hp.k_pool, device), storage_to_device(hp.cfg, hp.v_pool, device), device,
                   outer=[(lv.group_offsets, lv.length, lv.pages) for lv in hp.outer])

    def new_parts(self):
        g = self.geom
        o_part = torch.full((g.rows, g.n_parts, g.head_dim), float("nan"), dtype=torch.float32, device=self.device)
        lse_part = torch.full((g.rows, g.n_parts), float("nan"), dtype=torch.float32, device=self.device)
        return o_part, lse_part

    def decode(self, q: torch.Tensor, scale: Optional[float] = None, stream: int = 0):
        mc.mc_decode_attn(self.layout, q, self.cfg.scale if scale is None else scale, self.o, self.lse,
                          self.ws_ptr, self.ws_bytes, stream)
        return self.o, self.lse

    def close(self):
        if self.layout:
            mc.mc_kv_layout_destroy(self.layout)
            self.layout = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def make_device_problem(cfg: wl.Config, headroom_tokens: Optional[int] = None, device="cuda", outer=()
                        ) -> DeviceProblem:
    """Full-size instance whose pools are drawn on the device (torch's seeded generator) instead of being
    built on the host: lengths and page tables come from `workload`, every slot of both pools is N(0,1)
    rounded to the storage dtype, and K rows are turned into outliers with the configured probability."""
    prefix_len, suffix_len = wl.draw_lengths(cfg)
    tables = wl.build_page_tables(cfg, prefix_len, suffix_len, headroom_tokens)
    # outer cascade levels ((group_offsets, lengths) pairs) get fresh pages at the end of the pools
    outer_np = []
    for (go, lens) in outer:
        lens = np.asarray(lens, dtype=np.int32)
        npp = (lens.astype(np.int64) + cfg.page - 1) // cfg.page
        pages = np.full((len(lens), max(1, int(npp.max(initial=0)))), -1, dtype=np.int32)
        for j in range(len(lens)):
            pages[j, :int(npp[j])] = np.arange(tables.num_pages, tables.num_pages + int(npp[j]), dtype=np.int32)
            tables.num_pages += int(npp[j])
        outer_np.append((np.asarray(go, dtype=np.int32), lens, pages))
    tdtype = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    gen = torch.Generator(device=device)
    gen.manual_seed(cfg.seed * 1000003 + 17)
    shape = (tables.num_pages, cfg.Hkv, cfg.page, cfg.d)
    fp8 = cfg.dtype == "fp8"
    k_pool = torch.empty(shape, dtype=torch.uint8 if fp8 else tdtype, device=device)
    v_pool = torch.empty(shape, dtype=torch.uint8 if fp8 else tdtype, device=device)
    k_scale = torch.empty((tables.num_pages, cfg.Hkv), dtype=torch.float32, device=device) if fp8 else None
    v_scale = torch.empty((tables.num_pages, cfg.Hkv), dtype=torch.float32, device=device) if fp8 else None
    step = max(1, (1 << 28) // (cfg.Hkv * cfg.page * cfg.d))          # pages per chunk, bounds temporaries
    for lo in range(0, tables.num_pages, step):
        hi = min(tables.num_pages, lo + step)
        k = torch.empty((hi - lo,) + shape[1:], dtype=tdtype, device=device).normal_(generator=gen)
        v = torch.empty((hi - lo,) + shape[1:], dtype=tdtype, device=device).normal_(generator=gen)
        if cfg.k_outlier_prob > 0.0:
            mask = torch.rand((hi - lo, cfg.Hkv, cfg.page, 1), device=device, generator=gen) < cfg.k_outlier_prob
            k = torch.where(mask, k * cfg.k_outlier_scale, k)
        if fp8:
            # an input generator, not the library's quantiser: every page gets the scale its first token would have
            # given it (twice that row's largest magnitude over 448) and torch's cast makes the codes; whatever
            # lands in the pools IS the input, and the tests read it back from there
            for src, pool, sc in ((k, k_pool, k_scale), (v, v_pool, v_scale)):
                s = (src[:, :, 0].float().abs().amax(dim=-1) * 2.0 / 448.0).clamp_min(1e-30)
                sc[lo:hi] = s
                pool[lo:hi] = (src.float() / s[:, :, None, None]).clamp(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8)
        else:
            k_pool[lo:hi], v_pool[lo:hi] = k, v
        del k, v
    dp = DeviceProblem(cfg, tables, prefix_len, suffix_len, k_pool, v_pool, device, outer=outer_np,
                       k_scale=k_scale, v_scale=v_scale)
    dp.outer_np = outer_np
    return dp


def device_q(cfg: wl.Config, step: int, device="cuda") -> torch.Tensor:
    gen = torch.Generator(device=device)
    gen.manual_seed(cfg.seed * 7919 + 101 + step)
    tdtype = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    return torch.empty((cfg.B, cfg.Hq, cfg.d), dtype=tdtype, device=device).normal_(generator=gen)


def device_append(cfg: wl.Config, step: int, device="cuda"):
    gen = torch.Generator(device=device)
    gen.manual_seed(cfg.seed * 104729 + 211 + step)
    tdtype = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    k = torch.empty((cfg.B, cfg.Hkv, cfg.d), dtype=tdtype, device=device).normal_(generator=gen)
    v = torch.empty((cfg.B, cfg.Hkv, cfg.d), dtype=tdtype, device=device).normal_(generator=gen)
    return k, v


def logical_rows(dp: DeviceProblem, b: int, h: int, suffix_len_now: Optional[int] = None):
    """Copies candidate b's whole history for kv head h to the host, in token order, by plain indexing
    through the page tables: returns (K [n][d], V [n][d]) as float32 numpy arrays - for an e4m3 cache each of the
    two is a pair (codes uint8 [n][d], the scale of every token's page float32 [n]) instead."""
    j = int(np.searchsorted(dp.tables.group_offsets, b, side="right") - 1)
    P = int(dp.prefix_len[j].item())
    s = int(dp.suffix_len[b].item()) if suffix_len_now is None else suffix_len_now
    segments = []
    for (go, lens, pages) in getattr(dp, "outer_np", []):
        jo = int(np.searchsorted(go, b, side="right") - 1)
        segments.append((pages[jo], int(lens[jo])))
    segments += [(dp.tables.prefix_pages[j], P), (dp.tables.suffix_pages[b], s)]
    out, page = [], dp.cfg.page
    for pool, scale in ((dp.k_pool, dp.k_scale), (dp.v_pool, dp.v_scale)):
        parts, scales = [], []
        for pages_row, n in segments:
            n_pages = (n + page - 1) // page
            if n_pages:
                ids = torch.from_numpy(np.ascontiguousarray(pages_row[:n_pages], dtype=np.int64)).to(pool.device)
                rows = pool[ids, h].reshape(n_pages * page, -1)[:n]
                parts.append(rows.cpu().numpy() if pool.dtype == torch.uint8 else rows.float().cpu().numpy())
                if scale is not None:
                    scales.append(scale[ids, h].cpu().numpy().repeat(page)[:n])
        empty = np.zeros((0, dp.cfg.d), dtype=np.uint8 if pool.dtype == torch.uint8 else np.float32)
        rows = np.concatenate(parts, axis=0) if parts else empty
        if scale is not None:      # an e4m3 cache: the codes and each token's scale, for the caller to decode
            rows = (rows, np.concatenate(scales) if scales else np.zeros(0, dtype=np.float32))
        out.append(rows)
    return out[0], out[1]


class ScoringDeviceProblem:
    """A scoring problem on the device: every (sequence, position) is a candidate of a cascade layout whose base
    level is the shared prompts and whose one outer level is each sequence's own tokens under a causal row limit.
    Memory and marshalling only."""

    def __init__(self, hp: "wl.ScoringHostProblem", device="cuda", suffix_storage: bool = False):
        """suffix_storage: give the layout (empty) suffix tables, as a decode layout has, instead of none."""
        cfg = hp.cfg
        self.cfg, self.hp = cfg, hp
        i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)
        self.k_pool, self.v_pool = storage_to_device(cfg, hp.k_pool, device), storage_to_device(cfg, hp.v_pool, device)
        self.n_virtual = int(hp.seq_offsets[-1])
        Bv = max(1, self.n_virtual)
        self.t = {"go": i32(hp.group_offsets), "pp": i32(hp.prefix_pages), "pl": i32(hp.prefix_len),
                  "sp": i32(np.full((Bv, 1), -1)), "sl": i32(np.zeros(Bv)), "so": i32(hp.seq_offsets),
                  "qp": i32(hp.seq_pages), "ql": i32(hp.seq_len), "rl": i32(hp.row_limit)}
        d = mc.LayoutDesc()
        d.num_groups, d.batch, d.num_q_heads, d.num_kv_heads, d.head_dim = cfg.G, Bv, cfg.Hq, cfg.Hkv, cfg.d
        d.page_size, d.num_pages = wl.PAGE, hp.k_pool.shape[0]
        d.max_prefix_pages, d.max_suffix_pages = hp.prefix_pages.shape[1], 1 if suffix_storage else 0
        d.dtype = mc.MC_F32 if cfg.dtype == "f32" else mc.MC_BF16
        d.k_pool, d.v_pool = self.k_pool.data_ptr(), self.v_pool.data_ptr()
        d.group_offsets, d.prefix_pages, d.prefix_len = (self.t[k].data_ptr() for k in ("go", "pp", "pl"))
        if suffix_storage:
            d.suffix_pages, d.suffix_len = self.t["sp"].data_ptr(), self.t["sl"].data_ptr()
        lv = mc.PrefixLevel()
        lv.num_groups, lv.max_pages = cfg.B, hp.seq_pages.shape[1]
        lv.group_offsets, lv.pages, lv.len = (self.t[k].data_ptr() for k in ("so", "qp", "ql"))
        lv.row_limit = self.t["rl"].data_ptr()
        self.desc = d
        self.layout = mc.mc_kv_layout_create_cascade(d, [lv])
        self.geom = mc.mc_kv_layout_geometry(self.layout)
        self.ws_bytes = mc.mc_workspace_bytes(self.layout)
        self.ws = torch.empty(self.ws_bytes + 256, dtype=torch.uint8, device=device)
        self.ws_ptr = (self.ws.data_ptr() + 255) // 256 * 256
        tdtype = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
        self.o = torch.empty(Bv, cfg.Hq, cfg.d, dtype=tdtype, device=device)
        self.lse = torch.empty(Bv, cfg.Hq, dtype=torch.float32, device=device)

    def score(self, q: torch.Tensor, stream: int = 0):
        mc.mc_decode_attn(self.layout, q, self.cfg.scale, self.o, self.lse, self.ws_ptr, self.ws_bytes, stream)
        return self.o, self.lse

    def close(self):
        if self.layout:
            mc.mc_kv_layout_destroy(self.layout)
            self.layout = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
