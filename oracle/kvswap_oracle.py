"""CPU oracle for the KVSwap decode hot path -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

A plain, slow, float64 restatement of what the paper's predictor and the sparse decode
attention compute, one function per step, in the paper's order and notation.  It shares no
code with the CUDA library and must never be imported by it: only the tests, the smoke
check and the benchmark's CPU-baseline leg may call it.

Notation (Sec. 4.2, Sec. 4.3, App. A.2): N cached tokens, H_q query heads, H_k = H_kv KV
heads, d head dim, r metadata rank, A in R^{(H_k d) x r} the low-rank adapter with row block
A_g in R^{d x r} for KV head g, g(h) = floor(h / rho) the query-head -> KV-head map with
rho = H_q / H_kv, K_lr = Flatten(K) A the compressed K cache ("metadata"), G the group size,
M the number of selected groups.

Array conventions (all numpy, values already rounded to their storage type by the caller):
    K, V   [B, H_kv, N, d]        q   [B, H_q, d]        proj  [H_kv, d, r]  (A_g = proj[g])
    meta   [B, H_m, N, r]  with H_m = 1 (joint adapter, the paper's adopted design (b) of
           Sec. 4.2) or H_m = H_kv (one adapter per KV head, design (a) of Sec. 4.2)
    scope  "kv_head": one selection per (sequence, KV head), summing the rho query heads of
           that KV head;  "all_heads": one selection per sequence, summing all query heads
           (the paper's wording in Sec. 4.3, "Scoring and selection").

Pins (tests/test_oracle_pins.py): every function below is checked against something other
than itself -- exact rational arithmetic, closed forms, dense brute force, library-routine
special cases, hand-worked examples.  The one thing that has no pin is the *quality* of the
approximation (how much attention mass the selected groups capture): the paper prints no
number for the predictor alone, so that statistic is only reported -- "parity unpinned".
"""
from __future__ import annotations

import numpy as np

_STORE = {"f32": np.float32, "f16": np.float16, "f64": np.float64}  # "f64": no rounding (pins only)


def _rho(n_q_heads: int, n_kv_heads: int) -> int:
    if n_q_heads % n_kv_heads:
        raise ValueError("H_q must be a multiple of H_kv")
    return n_q_heads // n_kv_heads


# ------------------------------------------------------------------------------------------
# O1  K_lr = Flatten(K) A                                                       (Sec. 4.2)
# ------------------------------------------------------------------------------------------
def e4m3_decode_table() -> np.ndarray:
    """The 256 values of the 8-bit floating-point format E4M3 (1 sign, 4 exponent bits with bias 7,
    3 mantissa bits; no infinities; S.1111.111 is NaN; largest finite value 448; subnormals are
    multiples of 2^-9) -- the 8-bit storage format taken for the compact cache where the paper only
    says that its precision can be traded (Sec. 4.1, Sec. 4.2)."""
    vals = np.empty(256)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e, m = (code >> 3) & 0xF, code & 0x7
        if e == 0xF and m == 0x7:
            vals[code] = np.nan
        elif e == 0:
            vals[code] = sign * m * 2.0 ** -9
        else:
            vals[code] = sign * (8 + m) * 2.0 ** (e - 7 - 3)
    return vals


def e4m3_round(x: np.ndarray):
    """Nearest E4M3 value of every entry of x (float64): round to nearest, ties to the even
    mantissa, magnitudes beyond the largest finite value saturate to +-448.  Returns
    (values float64, codes uint8)."""
    x = np.asarray(x, dtype=np.float64)
    a = np.abs(x)
    _, ex = np.frexp(a)                                   # a = f * 2^ex, f in [0.5, 1)
    e = np.clip(ex - 1, -6, 8)                            # binade of a, clipped to the normal range
    quantum = np.ldexp(1.0, e - 3)                        # spacing of the format in that binade
    quantum = np.where(a < 2.0 ** -6, 2.0 ** -9, quantum)  # subnormal spacing below the smallest normal
    v = np.minimum(np.rint(a / quantum) * quantum, 448.0)   # np.rint rounds halves to even
    _, ex2 = np.frexp(v)
    e2 = np.clip(ex2 - 1, -6, 8)
    normal = v >= 2.0 ** -6
    mant = np.where(normal, v / np.ldexp(1.0, e2 - 3) - 8, v / 2.0 ** -9)
    code = np.where(normal, (e2 + 7) * 8, 0) + mant
    code = code.astype(np.int64) | np.where(np.signbit(x), 0x80, 0)
    return np.copysign(v, x), code.astype(np.uint8)


def project_keys(K: np.ndarray, proj: np.ndarray, meta_heads: int, meta_dtype: str = "f16",
                 meta_exp: int = 0) -> np.ndarray:
    """Compressed K cache.  Joint: meta[b,0,n,:] = sum_g K[b,g,n,:] A_g  (Flatten is head-major,
    column g*d+c <-> K[n,g,c]).  Per-head: meta[b,g,n,:] = K[b,g,n,:] A_g.
    The float64 result is rounded once, to nearest-even, into the storage type.  For the 8-bit
    type "e4m3" the stored value is round(K_lr * 2^-meta_exp) (returned as float32, which holds
    every E4M3 value exactly); the power of two only keeps the values inside the format's range
    and is multiplied back when the metadata is scored (`score_select(..., meta_exp=)`)."""
    K64 = K.astype(np.float64)
    A = proj.astype(np.float64)
    B, Hkv, N, d = K64.shape
    r = A.shape[2]
    if meta_heads == 1:
        meta = np.zeros((B, 1, N, r))
        for g in range(Hkv):
            meta[:, 0] += K64[:, g] @ A[g]
    elif meta_heads == Hkv:
        meta = np.empty((B, Hkv, N, r))
        for g in range(Hkv):
            meta[:, g] = K64[:, g] @ A[g]
    else:
        raise ValueError("meta_heads must be 1 or H_kv")
    if meta_dtype == "e4m3":
        return e4m3_round(np.ldexp(meta, -int(meta_exp)))[0].astype(np.float32)
    return meta.astype(_STORE[meta_dtype])


# ------------------------------------------------------------------------------------------
# O2  low-rank query  Q_h A_{g(h)}                                               (Eq. 1)
# ------------------------------------------------------------------------------------------
def lowrank_query(q: np.ndarray, proj: np.ndarray) -> np.ndarray:
    q64 = q.astype(np.float64)
    A = proj.astype(np.float64)
    B, Hq, d = q64.shape
    rho = _rho(Hq, A.shape[0])
    q_lr = np.empty((B, Hq, A.shape[2]))
    for h in range(Hq):
        q_lr[:, h] = q64[:, h] @ A[h // rho]
    return q_lr


# ------------------------------------------------------------------------------------------
# O3  per-head low-rank scores  (Q_h A_{g(h)}) K_lr^T                            (Eq. 1)
# ------------------------------------------------------------------------------------------
def head_scores(q_lr: np.ndarray, meta: np.ndarray, n_kv_heads: int) -> np.ndarray:
    """s[b,h,n]; raw logits (no softmax, no 1/sqrt(d): Eq. 1 approximates Q_h K^T itself)."""
    m64 = meta.astype(np.float64)
    B, Hq, r = q_lr.shape
    rho = _rho(Hq, n_kv_heads)
    Hm = m64.shape[1]
    s = np.empty((B, Hq, m64.shape[2]))
    for h in range(Hq):
        mh = 0 if Hm == 1 else h // rho
        s[:, h] = np.einsum("br,bnr->bn", q_lr[:, h], m64[:, mh])
    return s


# ------------------------------------------------------------------------------------------
# O4  one importance score per token: sum over heads      (Sec. 4.3, Scoring and selection)
# ------------------------------------------------------------------------------------------
def aggregate(s: np.ndarray, n_kv_heads: int, scope: str) -> np.ndarray:
    B, Hq, N = s.shape
    if scope == "all_heads":
        return s.sum(axis=1, keepdims=True)
    if scope == "kv_head":
        rho = _rho(Hq, n_kv_heads)
        return s.reshape(B, n_kv_heads, rho, N).sum(axis=2)
    raise ValueError("scope must be 'kv_head' or 'all_heads'")


# ------------------------------------------------------------------------------------------
# O5  ReduceMax over groups of G consecutive tokens                              (Sec. 4.3)
# ------------------------------------------------------------------------------------------
def pool(T: np.ndarray, G: int) -> np.ndarray:
    """R[b,s,j] = max_{0<=t<G} T[b,s,jG+t], j < floor(N/G).  The N mod G newest tokens form no
    complete group yet (rolling buffer, Sec. 4.4.1) and get no score."""
    B, S, N = T.shape
    NG = N // G
    return T[:, :, :NG * G].reshape(B, S, NG, G).max(axis=3)


# ------------------------------------------------------------------------------------------
# O6  TopK: the M highest-scoring groups                                         (Sec. 4.3)
# ------------------------------------------------------------------------------------------
def select(R: np.ndarray, M: int) -> np.ndarray:
    """Indices of the M' = min(M, NG) largest group scores of every (b, s) problem, where of
    two equal scores the lower index ranks first; returned sorted by index, shape [B,S,M']."""
    B, S, NG = R.shape
    Mp = min(M, NG)
    idx = np.empty((B, S, Mp), dtype=np.int32)
    for b in range(B):
        for s in range(S):
            order = sorted(range(NG), key=lambda j: (-R[b, s, j], j))
            idx[b, s] = np.sort(np.asarray(order[:Mp], dtype=np.int32))
    return idx


def score_select(q, proj, meta, G, M, scope="kv_head", head_softmax=False, meta_exp=0):
    """O2..O6 chained.  Returns (idx [B,S,M'], R [B,S,NG]).  With head_softmax the per-head scores
    pass through `softmax_over_context` before the head sum (the other reading of "attention
    scores" in Sec. 4.3).  `meta` holds the stored values of K_lr * 2^-meta_exp (meta_exp = 0 except
    for 8-bit metadata): the scores are those of meta * 2^meta_exp."""
    Hkv = proj.shape[0]
    if meta_exp:
        meta = np.ldexp(np.asarray(meta, dtype=np.float64), int(meta_exp))
    s = head_scores(lowrank_query(q, proj), meta, Hkv)
    if head_softmax:
        s = softmax_over_context(s, q.shape[2], G)
    R = pool(aggregate(s, Hkv, scope), G)
    return select(R, M), R


# ------------------------------------------------------------------------------------------
# O3'  variant: approximate attention weights instead of approximate logits
# ------------------------------------------------------------------------------------------
def softmax_over_context(s: np.ndarray, d: int, G: int) -> np.ndarray:
    """p[b,h,n] = softmax_n(s[b,h,n] / sqrt(d)) over the tokens of the complete groups,
    n < floor(N/G) G -- the weights exact attention would give them if the low-rank logits were
    exact and nothing else were attended.  Tokens of the open group keep no weight (0); they
    are dropped by `pool` anyway."""
    B, Hq, N = s.shape
    n_scored = (N // G) * G
    p = np.zeros_like(s, dtype=np.float64)
    if n_scored == 0:
        return p
    z = s[:, :, :n_scored].astype(np.float64) / np.sqrt(d)
    z = z - z.max(axis=2, keepdims=True)
    e = np.exp(z)
    p[:, :, :n_scored] = e / e.sum(axis=2, keepdims=True)
    return p


# ------------------------------------------------------------------------------------------
# O7  exact decode attention over the selected groups + rolling-buffer tail
#     (Sec. 4.4 decoding; Sec. 4.4.1 rolling buffer; Sec. 4.4.4 the three sources of entries)
# ------------------------------------------------------------------------------------------
def attend(q, K, V, idx, G, scope="kv_head", return_probs=False):
    """out[b,h,:] = sum_n p_n V[b,g(h),n,:],  p = softmax_n(q[b,h,:] . K[b,g(h),n,:] / sqrt(d))
    over the token set  U_{j in idx[b,s(h)]} [jG, jG+G)  U  [floor(N/G) G, N),
    s(h) = g(h) for scope 'kv_head', 0 for 'all_heads'.  Two-pass softmax with max subtraction.
    Also returns lse[b,h] = log sum_n exp(logit_n)."""
    q64, K64, V64 = q.astype(np.float64), K.astype(np.float64), V.astype(np.float64)
    B, Hq, d = q64.shape
    Hkv, N = K64.shape[1], K64.shape[2]
    rho = _rho(Hq, Hkv)
    NG = N // G
    out = np.empty((B, Hq, d))
    lse = np.empty((B, Hq))
    probs = {}
    for b in range(B):
        for h in range(Hq):
            g = h // rho
            s = g if scope == "kv_head" else 0
            tokens = [j * G + t for j in idx[b, s] for t in range(G)] + list(range(NG * G, N))
            tokens = np.asarray(tokens, dtype=np.int64)
            logits = (K64[b, g, tokens] @ q64[b, h]) / np.sqrt(d)
            mx = logits.max()
            e = np.exp(logits - mx)
            denom = e.sum()
            p = e / denom
            out[b, h] = p @ V64[b, g, tokens]
            lse[b, h] = mx + np.log(denom)
            if return_probs:
                probs[(b, h)] = (tokens, p)
    if return_probs:
        return out, lse, probs
    return out, lse


# ------------------------------------------------------------------------------------------
# O8  New KV entries: rolling buffer, flush of a completed group                 (Sec. 4.4.1)
# ------------------------------------------------------------------------------------------
def append_kv(K, V, meta, k_new, v_new, proj, G, meta_dtype="f16"):
    """One generated token joins the cache.  Its entries k_new, v_new [B, H_kv, d] are appended to
    the rolling buffer, i.e. become token N of K and V (the attention always covers the
    incomplete last group, see `attend`).  The predictor cannot rank them until their group is
    complete: only when the N+1 tokens end a group of G are the group's G rows compressed
    (O1) and appended to the compact cache.  `meta` holds rows of complete groups only,
    [B, H_m, floor(N/G) G, r]; H_m is taken from it.  Returns (K', V', meta', flushed)."""
    B, Hkv, N, d = K.shape
    if meta.shape[2] != (N // G) * G:
        raise ValueError("meta must hold exactly the rows of the complete groups")
    K2 = np.concatenate([K, k_new[:, :, None, :].astype(K.dtype)], axis=2)
    V2 = np.concatenate([V, v_new[:, :, None, :].astype(V.dtype)], axis=2)
    flushed = (N + 1) % G == 0
    if flushed:
        rows = project_keys(K2[:, :, N + 1 - G:N + 1], proj, meta.shape[1], meta_dtype)
        meta = np.concatenate([meta, rows.astype(meta.dtype)], axis=2)
    return K2, V2, meta, flushed


# ------------------------------------------------------------------------------------------
# O9  Reuse buffer: slots, slot table, FIFO replacement                          (Sec. 4.4.2)
# ------------------------------------------------------------------------------------------
def reuse_step(slot_group, head, selected):
    """One prediction step of one reuse buffer (one sequence and selection scope).

    slot_group[c] is the group id held by slot c (-1: empty) -- the paper's slot table; `head` is
    the FIFO position: slots are filled in the order 0, 1, .., C-1, 0, .., so the slot at `head`
    holds the group that was loaded longest ago.  `selected` lists the groups the predictor chose
    for this step (entries < 0 mean "no group" and get slot -1; a group listed twice is loaded once,
    by its first entry, and served to both).  In list order: a group
    found in the slot table is a hit and keeps its slot; any other group is loaded into the next
    slot in FIFO order, replacing what was there.  A slot that serves this step (a hit, or a
    group loaded earlier in the same step) is passed over by the FIFO position, since the
    attention of this step still reads it.

    Returns (slots, loads, slot_group', head'): slots[i] the slot serving selected[i]; loads the
    (group, slot) pairs fetched from the slow tier, in list order."""
    table = [int(x) for x in slot_group]
    C = len(table)
    groups = [int(j) for j in selected if j >= 0]
    if len(set(groups)) > C:
        raise ValueError("the reuse buffer must hold at least the groups of one step")
    wanted = set(groups)
    where = {g: c for c, g in enumerate(table) if g >= 0}
    busy = {where[g] for g in groups if g in where}          # slots of this step's hits
    slots, loads = [], []
    for j in selected:
        j = int(j)
        if j < 0:
            slots.append(-1)
        elif j in where:
            slots.append(where[j])
        else:
            while head in busy:
                head = (head + 1) % C
            old = table[head]
            if old >= 0:
                del where[old]
            table[head] = j
            where[j] = head
            busy.add(head)
            slots.append(head)
            loads.append((j, head))
            head = (head + 1) % C
    assert all(table[where[g]] == g for g in wanted)
    return slots, loads, table, head

