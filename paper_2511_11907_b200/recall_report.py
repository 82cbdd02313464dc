"""Recall of the low-rank predictor against exact scores, as a function of the rank r.

    python -m paper_2511_11907_b200.recall_report [--n-ctx 32768] [--ranks 8 16 32 64 128]

Keys with structure (Sec. 4.2 rests on the K cache being compressible): per KV head a latent of
`--latent` dimensions with a geometrically decaying spectrum, mixed into d channels, plus white
noise.  For each rank the adapter is taken from a calibration sample (top-r right singular
vectors), the compact cache is built with kvswap_project_keys and groups are selected with
kvswap_score_select; "exact" is the same sum -> group max -> top-M rule applied to the full q.K.
Reported: the share of the exact top-M groups that the predictor selects, and the share of each
head's softmax mass that the selected groups (plus the rolling-buffer tail) carry, next to what
the exact top-M groups carry.  A quality statistic on synthetic data -- nothing is asserted.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as kv
from . import device_workload as DW
from . import runtime as rt
from . import workloads as W


def structured_keys(gen, B, Hkv, N, d, latent, decay, noise):
    mix = torch.linalg.qr(torch.randn((Hkv, d, latent), generator=gen, device="cuda"))[0]        # [Hkv, d, latent]
    spectrum = decay ** torch.arange(latent, device="cuda", dtype=torch.float32)
    z = torch.randn((B, Hkv, N, latent), generator=gen, device="cuda") * spectrum
    K = torch.einsum("bgnl,gdl->bgnd", z, mix) * (d ** 0.5)
    return K + noise * torch.randn((B, Hkv, N, d), generator=gen, device="cuda"), mix


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--n-ctx", type=int, default=32768)
    ap.add_argument("--batch", type=int, default=2)
    ap.add_argument("--ranks", type=int, nargs="+", default=[8, 16, 32, 64, 128])
    ap.add_argument("--top-k", type=int, default=256)
    ap.add_argument("--group-size", type=int, default=8)
    ap.add_argument("--latent", type=int, default=48)
    ap.add_argument("--decay", type=float, default=0.9)
    ap.add_argument("--noise", type=float, default=0.15)
    ap.add_argument("--meta", choices=["joint", "per_head"], default="joint")
    a = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("recall_report needs a GPU: the library has no CPU path")
    B, Hq, Hkv, d, N, G, M = a.batch, 32, 8, 128, a.n_ctx, a.group_size, a.top_k
    rho, NG = Hq // Hkv, N // G
    gen = torch.Generator(device="cuda").manual_seed(20251111)
    Kf, mix = structured_keys(gen, B, Hkv, N, d, a.latent, a.decay, a.noise)
    K = Kf.to(torch.bfloat16).contiguous()                 # einsum results need not be dense in this order
    V = torch.randn((B, Hkv, N, d), generator=gen, device="cuda").to(torch.bfloat16)
    # queries that live mostly in the keys' subspace, as trained queries do
    zq = torch.randn((B, Hq, a.latent), generator=gen, device="cuda")
    q = (torch.einsum("bhl,hdl->bhd", zq, mix.repeat_interleave(rho, dim=0)) +
         0.3 * torch.randn((B, Hq, d), generator=gen, device="cuda")).to(torch.bfloat16).contiguous()
    # calibration sample: other tokens drawn by the same law (same mixing matrices)
    spectrum = a.decay ** torch.arange(a.latent, device="cuda", dtype=torch.float32)
    zc = torch.randn((8192, Hkv, a.latent), generator=gen, device="cuda") * spectrum
    calib = (torch.einsum("ngl,gdl->ngd", zc, mix) * (d ** 0.5) +
             a.noise * torch.randn((8192, Hkv, d), generator=gen, device="cuda")).contiguous()

    # exact rule: sum over the rho heads of a KV head, group max, top-M
    logits = torch.einsum("bgrd,bgnd->bgrn", q.float().view(B, Hkv, rho, d), K.float())        # [B, Hkv, rho, N]
    T = logits.sum(dim=2)[:, :, :NG * G].view(B, Hkv, NG, G).amax(dim=3)
    exact = T.topk(M, dim=2).indices
    probs = torch.softmax(logits / d ** 0.5, dim=3)                                             # per head

    def mass(groups):                                                                            # [B, Hkv, M] -> mean share
        tok = (groups.long().unsqueeze(-1) * G + torch.arange(G, device="cuda")).flatten(2)      # [B, Hkv, M G]
        sel = probs.gather(3, tok.unsqueeze(2).expand(B, Hkv, rho, tok.shape[2])).sum(dim=3)
        return float((sel + probs[:, :, :, NG * G:].sum(dim=3)).mean())

    mh = 1 if a.meta == "joint" else Hkv
    print(f"N = {N}, B = {B}, H_q/H_kv = {Hq}/{Hkv}, d = {d}, G = {G}, M = {M} ({100.0 * M / NG:.1f} % of the groups), "
          f"{a.meta} adapter, latent {a.latent}, decay {a.decay}, noise {a.noise}")
    print(f"softmax mass carried by the exact top-M groups: {mass(exact):.3f}")
    print("| rank r | compact cache / K cache | recall of the exact top-M groups | softmax mass carried |")
    print("|---|---|---|---|")
    for r in a.ranks:
        wl = W.Workload("recall", 3, 1, B, N, Hq, Hkv, d, r, G, M, W.BF16, W.F16, W.BF16, 8192)
        shape = rt.shape_for(wl, mh, W.SCOPE_KV_HEAD)
        proj = DW.adapter_on_device(calib, r, mh)
        ws, meta = rt.alloc_workspace(shape), rt.alloc_meta(shape)
        idx, nsel = rt.alloc_selection(shape)
        kv.kvswap_project_keys(shape, K, proj, meta, 0, N, ws)
        kv.kvswap_score_select(shape, q, proj, meta, idx, nsel, None, ws)
        torch.cuda.synchronize()
        hit = (idx.long().unsqueeze(3) == exact.unsqueeze(2)).any(dim=3).float().mean()
        ratio = mh * r * 2 / (Hkv * d * 2)
        print(f"| {r} | 1/{1 / ratio:.0f} | {float(hit):.3f} | {mass(idx):.3f} |")


if __name__ == "__main__":
    main()
