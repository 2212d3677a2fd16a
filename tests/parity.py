"""Helpers of the GPU-vs-oracle parity tests: tensor marshalling and the comparison protocol.

Protocol for keys.  The key quantizer rounds values that earlier roundings have corrected, so a
rounding tie resolved the other way (legitimate: both neighbours are nearest) changes everything
downstream of it in that token, and through the shared min/max possibly in its group.  Codes are
therefore compared like this: per group, find the earliest channel where GPU and oracle codes
differ; every differing element of that channel must be a tie in the oracle's own arithmetic
(|frac((x - zero)/scale) - 0.5| < 1e-5 at 2 bits; the same fraction of the group's RANGE at other bit
widths, i.e. 1e-5 * L/3 in code units, because the float32 error of the corrected value does not shrink
when the grid gets finer) and differ by exactly one level; force the GPU's choice
there, re-run the oracle on that group, repeat.  The run passes iff every forced decision was such
a tie and nothing differs afterwards.  The raw (pre-replay) identical fraction is reported too and
must be >= 99.9 %.  Every forced tie's distance from the midpoint is kept, so that a report can say how
many of them lie outside the literal 1e-5 code units (possible only at more than 2 bits).

The projected error is checked on both readings of "the subspace basis": the objective's own weighting
||Qhat (k - khat)||_F (rows of Qhat = sigma_i v_i) and the orthonormal basis ||V_r^T (k - khat)||_F
(rows of Qhat normalised), each within 1e-3 relative of the oracle's.
"""
import numpy as np
import torch

import oracle
import squat_inputs as si

TIE_BAND = 1e-5          # in code units at 2 bits (L = 3); scaled by L/3 for other bit widths


def to_torch(a: np.ndarray, dtype: str, device="cuda") -> torch.Tensor:
    """Generator output (float32 array or uint16 bf16 bit patterns) -> torch tensor on device."""
    if dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(a)).to(device)
    t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
    return t.to(device)


def from_torch_bf16(t: torch.Tensor) -> np.ndarray:
    """torch bf16 tensor -> float32 numpy, exact."""
    return si.bf16_bits_to_f32(t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16))


def stacked_queries(cfg, h, n_tokens=None) -> np.ndarray:
    """Rows = all prompt tokens of the query heads feeding KV head h (float64, exact widening)."""
    qs = [si.to_f32(si.gen_queries_head(cfg, hq, n_tokens), cfg.dtype)
          for hq in range(h * cfg.q_per_kv, (h + 1) * cfg.q_per_kv)]
    return np.concatenate(qs, axis=0).astype(np.float64)


def oracle_mats(cfg, h, n_tokens=None, rank_r=None, lam=None, g=None):
    return oracle.build_W(stacked_queries(cfg, h, n_tokens), cfg.rank_r if rank_r is None else rank_r,
                          cfg.lam if lam is None else lam, cfg.block_g if g is None else g)


def alloc_key_outputs(B, H, T, d, bits, G, device="cuda"):
    codes = torch.empty((B, H, T, d * bits // 8), dtype=torch.uint8, device=device)
    scales = torch.empty((B, H, T // G, d), dtype=torch.float32, device=device)
    zeros = torch.empty((B, H, T // G, d), dtype=torch.float32, device=device)
    return codes, scales, zeros


def alloc_value_outputs(B, H, T, d, bits, G, device="cuda"):
    codes = torch.empty((B, H, T, d * bits // 8), dtype=torch.uint8, device=device)
    scales = torch.empty((B, H, T, d // G), dtype=torch.float32, device=device)
    zeros = torch.empty((B, H, T, d // G), dtype=torch.float32, device=device)
    return codes, scales, zeros


def _projection_checks(stats, gpu_deq, final_khat, K64, Qhat):
    """Relative differences of the projected errors (GPU against oracle) on Qhat and on the orthonormal V_r."""
    if Qhat is None or Qhat.shape[0] == 0:
        return
    norms = np.linalg.norm(Qhat, axis=1)
    Vr = Qhat[norms > 0] / norms[norms > 0][:, None]           # rows v_i: Qhat = diag(sigma) V_r^T
    dg, do = gpu_deq.astype(np.float64) - K64, final_khat - K64
    for name, basis in (("proj_rel", Qhat), ("proj_rel_vr", Vr)):
        pg, po = np.linalg.norm(dg @ basis.T), np.linalg.norm(do @ basis.T)
        stats[name] = float(abs(pg - po) / po)
        assert abs(pg - po) <= 1e-3 * po, (name, pg, po)


def compare_key_unit(K64, W64, G, bits, gpu_codes, gpu_scale, gpu_zero, gpu_deq=None, Qhat=None, max_replays=64,
                     meta16=False):
    """Compares one (batch, head) unit.  K64 [n,d] float64; gpu_codes [n,d] unpacked uint8;
    gpu_scale/zero [n/G, d] float32; gpu_deq [n,d] float32 (optional).  Returns a dict of statistics;
    raises AssertionError with a precise message on any violation of the protocol.
    meta16: the cache stores scale and zero-point as binary16 (gpu_scale / gpu_zero hold those values widened to
    float32); see compare_key_unit_meta16."""
    if meta16:
        return compare_key_unit_meta16(K64, W64, G, bits, gpu_codes, gpu_scale, gpu_zero, gpu_deq, Qhat, max_replays)
    n, d = K64.shape
    base = oracle.quant_keys(K64, G, bits, W64, want_tval=True)
    raw_equal = int((base["codes"] == gpu_codes).sum())
    ties = 0
    tie_dist = []
    final_codes = base["codes"].copy()
    final_khat = base["Khat"].copy()
    final_scale, final_zero = base["scale"].copy(), base["zero"].copy()
    bad_groups = np.unique(np.nonzero(base["codes"] != gpu_codes)[0] // G)
    for grp in bad_groups:
        lo, hi = grp * G, (grp + 1) * G
        force = -np.ones((G, d), dtype=np.int16)
        o = {k: v[lo:hi] if k in ("codes", "Khat", "tval") else v[grp:grp + 1] for k, v in base.items()}
        for _ in range(max_replays):
            diff = o["codes"] != gpu_codes[lo:hi]
            if not diff.any():
                break
            j0 = int(np.nonzero(diff.any(axis=0))[0][0])
            for i in np.nonzero(diff[:, j0])[0]:
                t = o["tval"][i, j0]
                frac = abs((t - np.floor(t)) - 0.5)
                cg, co = int(gpu_codes[lo + i, j0]), int(o["codes"][i, j0])
                assert abs(cg - co) == 1 and frac < TIE_BAND * ((1 << bits) - 1) / 3.0, (
                    f"non-tie mismatch: group {grp} token {i} channel {j0}: gpu {cg} oracle {co} "
                    f"t={t!r} |frac-0.5|={frac:.3e}")
                force[i, j0] = cg
                ties += 1
                tie_dist.append(float(frac))
            o = oracle.quant_keys(K64[lo:hi], G, bits, W64, force=force, want_tval=True)
        else:
            raise AssertionError(f"group {grp}: replay did not converge")
        final_codes[lo:hi] = o["codes"]
        final_khat[lo:hi] = o["Khat"]
        final_scale[grp], final_zero[grp] = o["scale"][0], o["zero"][0]
    assert np.array_equal(final_codes, gpu_codes)
    stats = {"elements": n * d, "raw_equal": raw_equal, "ties": ties, "raw_fraction": raw_equal / (n * d),
             "ties_beyond_1e-5": sum(1 for f in tie_dist if f >= TIE_BAND), "max_tie_dist": max(tie_dist, default=0.0)}
    # scale / zero: float32 roundings of fp64 vs fp32 working values
    sc_err = np.abs(gpu_scale.astype(np.float64) - final_scale).max() / max(np.abs(final_scale).max(), 1e-30)
    zr_err = np.abs(gpu_zero.astype(np.float64) - final_zero).max() / max(np.abs(final_zero).max(), 1e-30)
    stats["scale_rel_err"], stats["zero_rel_err"] = float(sc_err), float(zr_err)
    assert sc_err < 1e-4 and zr_err < 1e-4, (sc_err, zr_err)
    if gpu_deq is not None:
        rel = np.linalg.norm(gpu_deq.astype(np.float64) - final_khat) / np.linalg.norm(final_khat)
        stats["deq_rel_fro"] = float(rel)
        assert rel < 1e-3, rel
        _projection_checks(stats, gpu_deq, final_khat, K64, Qhat)
    return stats


META_TIE_BAND = 1e-5     # a binary16 rounding of scale / zero counts as a tie within this fraction of the value's size


def compare_key_unit_meta16(K64, W64, G, bits, gpu_codes, gpu_scale, gpu_zero, gpu_deq=None, Qhat=None, max_replays=64):
    """The protocol of compare_key_unit for the 16-bit-metadata cache.  Besides rounding ties of codes there are
    rounding ties of the metadata: the float32 scale or zero-point of a (group, channel) lies so close to the middle
    between two binary16 numbers that the float64 oracle and the float32 kernel, whose corrected values differ by
    rounding noise, store different neighbours.  Such a pair is accepted if the kernel's value is the adjacent
    binary16 number and the oracle's unrounded value lies within META_TIE_BAND (relative to |zero| + range) of the
    midpoint; the kernel's stored value is then forced into the oracle and the group replayed, exactly as for codes.
    At the end codes, scales and zero-points must be identical."""
    n, d = K64.shape
    L = (1 << bits) - 1
    base = oracle.quant_keys(K64, G, bits, W64, want_tval=True, meta16=True)
    raw_equal = int((base["codes"] == gpu_codes).sum())
    ties = meta_ties = 0
    tie_dist = []
    final_codes, final_khat = base["codes"].copy(), base["Khat"].copy()
    final_scale, final_zero = base["scale"].copy(), base["zero"].copy()
    code_bad = np.nonzero(base["codes"] != gpu_codes)[0] // G
    meta_bad = np.nonzero((base["scale"] != gpu_scale) | (base["zero"] != gpu_zero))[0]
    for grp in np.unique(np.concatenate([code_bad, meta_bad])):
        lo, hi = grp * G, (grp + 1) * G
        force = -np.ones((G, d), dtype=np.int16)
        fs = np.full((1, d), np.nan, np.float32)
        fz = np.full((1, d), np.nan, np.float32)
        keys = ("codes", "Khat", "tval")
        o = {k: (v[lo:hi] if k in keys else v[grp:grp + 1]) for k, v in base.items()}
        for _ in range(max_replays):
            cdiff = (o["codes"] != gpu_codes[lo:hi]).any(axis=0)
            mdiff = (o["scale"][0] != gpu_scale[grp]) | (o["zero"][0] != gpu_zero[grp])
            if not cdiff.any() and not mdiff.any():
                break
            j0 = int(np.nonzero(cdiff | mdiff)[0][0])
            if mdiff[j0]:
                size = abs(float(o["raw_zero"][0, j0])) + L * abs(float(o["raw_scale"][0, j0]))
                for name, store, raw, gpu in (("scale", fs, o["raw_scale"][0, j0], gpu_scale[grp, j0]),
                                              ("zero", fz, o["raw_zero"][0, j0], gpu_zero[grp, j0])):
                    ora = o[name][0, j0]
                    if ora == gpu:
                        continue
                    h_or, h_gpu = np.float16(ora), np.float16(gpu)
                    assert np.float32(h_gpu) == gpu, f"stored {name} is not a binary16 number: {gpu!r}"
                    step = np.nextafter(h_or, h_gpu)
                    mid = 0.5 * (float(ora) + float(gpu))
                    assert step == h_gpu and abs(float(raw) - mid) <= META_TIE_BAND * size, (
                        f"metadata mismatch that is no tie: group {grp} channel {j0} {name}: gpu {gpu!r} oracle {ora!r} "
                        f"unrounded {float(raw)!r} midpoint {mid!r}")
                    store[0, j0] = gpu
                    meta_ties += 1
            else:
                diff = o["codes"][:, j0] != gpu_codes[lo:hi, j0]
                for i in np.nonzero(diff)[0]:
                    t = o["tval"][i, j0]
                    frac = abs((t - np.floor(t)) - 0.5)
                    cg, co = int(gpu_codes[lo + i, j0]), int(o["codes"][i, j0])
                    assert abs(cg - co) == 1 and frac < TIE_BAND * L / 3.0, (
                        f"non-tie mismatch: group {grp} token {i} channel {j0}: gpu {cg} oracle {co} "
                        f"t={t!r} |frac-0.5|={frac:.3e}")
                    force[i, j0] = cg
                    ties += 1
                    tie_dist.append(float(frac))
            o = oracle.quant_keys(K64[lo:hi], G, bits, W64, force=force, want_tval=True, meta16=True, force_meta=(fs, fz))
        else:
            raise AssertionError(f"group {grp}: replay did not converge")
        final_codes[lo:hi], final_khat[lo:hi] = o["codes"], o["Khat"]
        final_scale[grp], final_zero[grp] = o["scale"][0], o["zero"][0]
    assert np.array_equal(final_codes, gpu_codes)
    assert np.array_equal(final_scale, gpu_scale) and np.array_equal(final_zero, gpu_zero)
    stats = {"elements": n * d, "raw_equal": raw_equal, "ties": ties, "meta_ties": meta_ties,
             "raw_fraction": raw_equal / (n * d),
             "ties_beyond_1e-5": sum(1 for f in tie_dist if f >= TIE_BAND), "max_tie_dist": max(tie_dist, default=0.0)}
    if gpu_deq is not None:
        rel = np.linalg.norm(gpu_deq.astype(np.float64) - final_khat) / np.linalg.norm(final_khat)
        stats["deq_rel_fro"] = float(rel)
        assert rel < 1e-3, rel
        _projection_checks(stats, gpu_deq, final_khat, K64, Qhat)
    return stats


def rtn_per_channel_f32(K32, G, bits):
    """Per-channel round-to-nearest over groups of G tokens in binary32, through the oracle's
    per-token routine applied to the transposed groups."""
    n, d = K32.shape
    codes = np.empty((n, d), dtype=np.uint8)
    scale = np.empty((n // G, d), dtype=np.float32)
    zero = np.empty((n // G, d), dtype=np.float32)
    for grp in range(n // G):
        blk = np.ascontiguousarray(K32[grp * G:(grp + 1) * G].T)      # [d, G]
        o = oracle.quant_values_f32(blk, G, bits)
        codes[grp * G:(grp + 1) * G] = o["codes"].T
        scale[grp], zero[grp] = o["scale"][:, 0], o["zero"][:, 0]
    return codes, scale, zero
