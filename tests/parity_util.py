"""Comparators between the CUDA library and the CPU oracle, and the glue that runs one layer
through the C ABI.  The tolerances are the ones the parity tests assert."""
import numpy as np
import torch

from oracle import kvswap_oracle as O
from paper_2511_11907_b200 import binding as kv
from paper_2511_11907_b200 import runtime as rt
from paper_2511_11907_b200 import workloads as W

SCOPE_NAME = {W.SCOPE_KV_HEAD: "kv_head", W.SCOPE_ALL_HEADS: "all_heads"}
META_NAME = {W.F32: "f32", W.F16: "f16"}

# Attention output / lse: absolute bounds per K/V storage type.
OUT_ATOL = {W.F32: 1e-5, W.BF16: 2e-2, W.F16: 2e-2}
# With identical stored inputs on both sides only fp32 accumulation differs, so the observed
# error is orders of magnitude below the 16-bit bound; this tighter figure catches regressions.
OUT_ATOL_TIGHT = {W.F32: 1e-5, W.BF16: 1e-4, W.F16: 1e-4}
SELECT_BAND = 1e-5            # relative width of the tie band around the M'-th score


def f16_ulp(x):
    """Spacing of binary16 at |x| (normal or subnormal)."""
    ax = np.abs(np.asarray(x, dtype=np.float64))
    e = np.floor(np.log2(np.maximum(ax, 2.0 ** -14)))
    return 2.0 ** (e - 10)


def project_tolerance(K, proj, meta_heads, oracle_meta, meta_dtype):
    """|gpu - oracle| bound for the metadata: one unit in the last place of the storage type (the
    GPU rounds an fp32 sum, the oracle an exact one) plus the fp32 accumulation error, taken as
    2^-21 * sum_c |K||A| (about n*2^-24 for the n <= 1024 terms summed, with margin)."""
    absK, absA = np.abs(K.astype(np.float64)), np.abs(proj.astype(np.float64))
    per_head = np.einsum("bgnc,gcr->bgnr", absK, absA)
    absdot = per_head.sum(axis=1, keepdims=True) if meta_heads == 1 else per_head
    om = oracle_meta.astype(np.float64)
    ulp = f16_ulp(om) if meta_dtype == W.F16 else np.abs(om) * 2.0 ** -23
    return ulp + 2.0 ** -21 * absdot


def check_selection(R, idx_gpu, nsel_gpu, M, select_band=None):
    """The selection comparator: bit-exact group selection except inside the tie band.
    R: oracle group scores [B,S,NG]; idx_gpu [B,S,M]; nsel_gpu [B,S].  Returns #problems that had
    more than one group inside the band.  select_band overrides the relative width of the band."""
    rel_band = SELECT_BAND if select_band is None else select_band
    B, S, NG = R.shape
    Mp = min(M, NG)
    ambiguous_problems = 0
    idx_o = O.select(R, M)
    for b in range(B):
        for s in range(S):
            assert nsel_gpu[b, s] == Mp
            got = idx_gpu[b, s, :Mp]
            assert np.all(idx_gpu[b, s, Mp:] == -1)
            assert np.all(got >= 0) and np.all(got < NG)
            assert np.all(np.diff(got) > 0), "indices must be ascending and distinct"
            if Mp == 0:
                continue
            tau = np.sort(R[b, s])[::-1][Mp - 1]
            band = rel_band * max(abs(tau), 1e-30)
            amb = np.abs(R[b, s] - tau) <= band
            must = np.flatnonzero((R[b, s] > tau) & ~amb)
            never = np.flatnonzero((R[b, s] < tau) & ~amb)
            gs = set(got.tolist())
            assert set(must.tolist()) <= gs, "a clearly better group is missing"
            assert not (set(never.tolist()) & gs), "a clearly worse group was selected"
            if amb.sum() == 1:
                assert np.array_equal(got, idx_o[b, s]), "no tie: selection must be bit-exact"
            else:
                ambiguous_problems += 1
    return ambiguous_problems


def check_scores(R_oracle, R_gpu, absdot_max):
    """Group scores: 1e-5 relative plus the fp32 accumulation floor 4e-6 * max_n sum_i |u_i m_ni|
    (absdot_max [B,S], from the oracle's quantities)."""
    tol = 1e-5 * np.abs(R_oracle) + 4e-6 * absdot_max[:, :, None] + 1e-6
    err = np.abs(R_gpu.astype(np.float64) - R_oracle)
    assert np.all(err <= tol), f"group score error {err.max():.3e} exceeds tolerance"


def oracle_score_parts(li, meta_values, scope):
    """Oracle R and the magnitude bound used by check_scores."""
    Hkv = li.wl.n_kv_heads
    q_lr = O.lowrank_query(li.q, li.proj)
    s = O.head_scores(q_lr, meta_values, Hkv)
    T = O.aggregate(s, Hkv, SCOPE_NAME[scope])
    R = O.pool(T, li.wl.group_size)
    Tabs = O.aggregate(O.head_scores(np.abs(q_lr), np.abs(meta_values.astype(np.float64)), Hkv), Hkv,
                       SCOPE_NAME[scope])
    return R, Tabs.max(axis=2)


class DeviceLayer:
    """One layer's inputs on the GPU plus the buffers the three calls need."""

    def __init__(self, li: W.LayerInputs, scope=W.SCOPE_KV_HEAD, **shape_override):
        wl = li.wl
        self.li = li
        self.shape = rt.shape_for(wl, li.meta_heads, scope, **shape_override)
        self.K = rt.to_device(li.K_raw, wl.kv_dtype)
        self.V = rt.to_device(li.V_raw, wl.kv_dtype)
        self.q = rt.to_device(li.q_raw, wl.q_dtype)
        self.proj = torch.from_numpy(np.ascontiguousarray(li.proj, dtype=np.float32)).cuda()
        self.ws = rt.alloc_workspace(self.shape)
        self.meta = rt.alloc_meta(self.shape)
        self.idx, self.nsel = rt.alloc_selection(self.shape)
        self.out, self.lse = rt.alloc_output(self.shape)
        self.scores = torch.empty((wl.batch, self.shape.n_scopes, max(self.shape.n_groups, 1)),
                                  dtype=torch.float32, device="cuda")

    def poison(self):
        """Fill every output and the workspace with NaN / garbage so unwritten results show."""
        self.ws.fill_(0xFF)
        kv.kvswap_workspace_init(self.ws)
        self.meta.fill_(float("nan"))
        self.idx.fill_(-7)
        self.nsel.fill_(-7)
        self.out.fill_(float("nan"))
        self.lse.fill_(float("nan"))
        self.scores.fill_(float("nan"))

    def project(self, n_begin=0, n_end=None):
        kv.kvswap_project_keys(self.shape, self.K, self.proj, self.meta, n_begin,
                               self.shape.n_ctx if n_end is None else n_end, self.ws)
        torch.cuda.synchronize()
        return rt.to_host_f32(self.meta)

    def set_meta(self, meta_np):
        """Load oracle metadata (numpy float16/float32 array) into the device buffer."""
        if self.shape.meta_dtype == W.F16:
            self.meta.copy_(torch.from_numpy(np.ascontiguousarray(meta_np).view(np.int16)).view(torch.float16))
        else:
            self.meta.copy_(torch.from_numpy(np.ascontiguousarray(meta_np, dtype=np.float32)))

    def score_select(self, q=None, with_scores=True):
        kv.kvswap_score_select(self.shape, self.q if q is None else q, self.proj, self.meta, self.idx, self.nsel,
                               self.scores if with_scores else None, self.ws)
        torch.cuda.synchronize()
        return self.idx.cpu().numpy(), self.nsel.cpu().numpy(), self.scores.cpu().numpy()

    def set_selection(self, idx_np, nsel=None):
        B, S, M = self.idx.shape
        full = np.full((B, S, M), -1, dtype=np.int32)
        full[:, :, :idx_np.shape[2]] = idx_np
        self.idx.copy_(torch.from_numpy(full))
        n = np.full((B, S), idx_np.shape[2], dtype=np.int32) if nsel is None else np.asarray(nsel, dtype=np.int32)
        self.nsel.copy_(torch.from_numpy(n))

    def sparse_decode(self, with_lse=True):
        kv.kvswap_sparse_decode(self.shape, self.q, self.K, self.V, self.idx, self.nsel, self.out,
                                self.lse if with_lse else None, self.ws)
        torch.cuda.synchronize()
        return self.out.cpu().numpy(), self.lse.cpu().numpy()
