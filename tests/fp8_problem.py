"""Test helper: turns a host problem (logical K/V per group and candidate, page tables) into an e4m3 cache image
with per-(page, kv head) scales, using the ORACLE's quantiser (oracle/fp8.py) - test infrastructure, never imported
by the library.  The logical views become the values the codes stand for (float64), which is what the attention
oracle is given; `append` mirrors mc_kv_append on the host so that codes and scales can be compared bit for bit."""
import numpy as np

from oracle import fp8
from paper_2601_05475_b200 import workload as wl

FILL_CODE = 0x7E        # +448: the largest finite code, in every slot no sequence owns
FILL_SCALE = 25.0       # ... times this scale = 11200: finite and far outside the data


class Fp8HostProblem:
    def __init__(self, hp: wl.HostProblem):
        cfg = hp.cfg
        assert cfg.dtype == "fp8"
        self.hp, self.cfg, self.tables = hp, cfg, hp.tables
        n_pages = hp.tables.num_pages
        self.k_pool = np.full((n_pages, cfg.Hkv, wl.PAGE, cfg.d), FILL_CODE, dtype=np.uint8)
        self.v_pool = self.k_pool.copy()
        self.k_scale = np.full((n_pages, cfg.Hkv), FILL_SCALE, dtype=np.float32)
        self.v_scale = self.k_scale.copy()
        self.prefix_len, self.suffix_len = hp.prefix_len.copy(), hp.suffix_len.copy()
        self.k_prefix = [self._store(hp.k_prefix[j], hp.tables.prefix_pages[j], self.k_pool, self.k_scale) for j in range(cfg.G)]
        self.v_prefix = [self._store(hp.v_prefix[j], hp.tables.prefix_pages[j], self.v_pool, self.v_scale) for j in range(cfg.G)]
        self.k_suffix = [self._store(hp.k_suffix[b], hp.tables.suffix_pages[b], self.k_pool, self.k_scale) for b in range(cfg.B)]
        self.v_suffix = [self._store(hp.v_suffix[b], hp.tables.suffix_pages[b], self.v_pool, self.v_scale) for b in range(cfg.B)]
        self.outer = []
        for lv in hp.outer:
            k = [self._store(lv.k[j], lv.pages[j], self.k_pool, self.k_scale) for j in range(len(lv.length))]
            v = [self._store(lv.v[j], lv.pages[j], self.v_pool, self.v_scale) for j in range(len(lv.length))]
            self.outer.append((k, v, lv.group_offsets.tolist()))

    @staticmethod
    def _store(tokens, pages_row, pool, scale):
        """Quantises one sequence page by page, writes codes and scales through the page-table row, returns the values
        the codes stand for, [n][Hkv][d] float64."""
        n = tokens.shape[0]
        codes, sc = fp8.quantise_sequence(tokens)
        for pg in range((n + wl.PAGE - 1) // wl.PAGE):
            lo, hi = pg * wl.PAGE, min(n, (pg + 1) * wl.PAGE)
            pid = int(pages_row[pg])
            pool[pid, :, :hi - lo, :] = np.transpose(codes[lo:hi], (1, 0, 2))
            scale[pid] = sc[pg]
        return fp8.dequantise_sequence(codes, sc)

    def append_one(self, b, k_row, v_row):
        """One token of candidate b (k_row, v_row [Hkv][d]), as the library stores it: slot 0 of a page fixes the
        page's scales."""
        s = int(self.suffix_len[b])
        pid, slot = int(self.tables.suffix_pages[b, s // wl.PAGE]), s % wl.PAGE
        for new, pool, scale, logical in ((k_row, self.k_pool, self.k_scale, self.k_suffix),
                                          (v_row, self.v_pool, self.v_scale, self.v_suffix)):
            row = np.zeros((1, self.cfg.Hkv, self.cfg.d), dtype=np.float64)
            for h in range(self.cfg.Hkv):
                if slot == 0:
                    scale[pid, h] = fp8.page_scale(new[h])
                pool[pid, h, slot] = fp8.quantise_rows(new[h][None], scale[pid, h])[0]
                row[0, h] = fp8.dequantise(pool[pid, h, slot], scale[pid, h])
            logical[b] = np.concatenate([logical[b], row], axis=0)
        self.suffix_len[b] = s + 1

    def append(self, k_new, v_new):
        """One token per candidate (k_new, v_new [B][Hkv][d]), as mc_kv_append stores it."""
        for b in range(self.cfg.B):
            self.append_one(b, k_new[b], v_new[b])


def make(cfg: wl.Config, outer=(), **kw) -> Fp8HostProblem:
    hp = wl.make_host_problem(cfg, **kw)
    for i, (go, lens) in enumerate(outer):
        wl.add_outer_level(hp, go, lens, i)
    return Fp8HostProblem(hp)
