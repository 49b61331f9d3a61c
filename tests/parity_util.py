"""Lock-step comparison of the CUDA library with the CPU oracle.

Direction of data: the oracle's state is imported INTO the CUDA layer before each
compared chunk; nothing computed by the CUDA path is ever fed to the oracle.
"""

from __future__ import annotations

import numpy as np
import torch

from oracle import locret_oracle as O

ATTN_TOL = 2e-2       # |delta| <= ATTN_TOL * max(1, |ref|) + (P_ULP + V_ULP) * sum_i p_i |v_i| + flip_sens
P_ULP = 2.0 ** -8     # the probabilities enter the second contraction as bf16 operands
V_ULP = 2.0 ** -7     # a stored V element may round to either bf16 neighbour (fp32 vs fp64 sum)
SCORE_TOL = 1e-2      # |delta| <= SCORE_TOL * max(|ref|, rms(ref over the chunk))
BAND = 1e-2           # index sets must agree outside this band around the cut
FLIP_FRACTION = 5e-3  # share of stored chunk K/V elements allowed to sit one bf16 ulp apart (measured 2.3e-3 at K = 4096)


def bf16_dev(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).cuda()


def make_pair(shape, weights, budget, chunk, n_stab, reserve=0):
    from paper_2410_01805_b200 import LocretLayer
    wqkv, w1, w2 = weights
    ora = O.OracleLayer(shape, wqkv, w1, w2, budget, chunk, n_stab, reserve=reserve, mirror=True)
    ora.want_flip_sens = True
    gpu = LocretLayer(shape, bf16_dev(wqkv), bf16_dev(w1), bf16_dev(w2), budget, chunk, n_stab,
                      reserve=reserve)
    return ora, gpu


def check_attention(got: np.ndarray, ref: np.ndarray, what="", abs_ref=None, flip_sens=None):
    """abs_ref = sum_i p_i |v_i| from the oracle: rows that attend to outlier tokens sum terms
    far larger than their result; a bf16 probability operand carries up to 2^-9 relative error
    per term, and a value element whose exact projection lies next to a bf16 rounding boundary
    may be stored one ulp apart by the two sides (checked separately), which moves the output
    by up to p_i * ulp(v_i).  Without abs_ref the bound is the plain mixed absolute/relative one."""
    ok = ~np.isnan(ref)
    err = np.abs(got[ok] - ref[ok])
    bound = ATTN_TOL * np.maximum(1.0, np.abs(ref[ok]))
    if abs_ref is not None:
        bound = bound + (P_ULP + V_ULP) * abs_ref[ok]
    if flip_sens is not None:
        # stored Q/K elements may also sit one ulp apart (same cause); flip_sens is the oracle's
        # first-order propagation of one such flip per key into the output
        bound = bound + flip_sens[ok]
    worst = float(np.max(err / bound)) if err.size else 0.0
    assert worst <= 1.0, f"{what} attention: worst err/bound {worst:.3f}, max abs {err.max():.4g}"
    return float(err.max()) if err.size else 0.0


def check_scores(got: np.ndarray, ref: np.ndarray, what=""):
    rms = np.sqrt(np.mean(ref ** 2, axis=0, keepdims=True))
    bound = SCORE_TOL * np.maximum(np.abs(ref), rms) + 1e-30
    worst = float(np.max(np.abs(got - ref) / bound))
    assert worst <= 1.0, f"{what} scores: worst err/bound {worst:.3f}"
    return worst


def check_keep_band(kept_slots, s_ref, budget, n_prot, oracle_keep, what="", n_pre=0):
    """kept_slots: ascending slot indices (into cache ‖ chunk) kept by the CUDA path for one head.
    n_pre: protected prefix of the query-aware variant (0 = Algorithm 1)."""
    n = len(s_ref)
    kept = np.zeros(n, dtype=bool)
    kept[kept_slots] = True
    assert kept.sum() == min(budget, n), f"{what}: kept {kept.sum()} units"
    assert kept[n - n_prot:].all(), f"{what}: a protected unit was evicted"
    assert kept[:n_pre].all(), f"{what}: a unit of the protected prefix was evicted"
    rest = n - n_prot
    k = budget - n_prot - n_pre
    if k == 0:
        assert not kept[n_pre:rest].any()
        return True
    if k >= rest - n_pre:
        return True
    sr = np.where(np.isnan(s_ref[n_pre:rest]), -np.inf, s_ref[n_pre:rest])
    srt = np.sort(sr)[::-1]
    tau_hi, tau_lo = srt[k - 1], srt[k]
    must = sr >= tau_hi + BAND
    never = sr <= tau_lo - BAND
    assert kept[n_pre:rest][must].all(), f"{what}: a unit above the band was evicted"
    assert not kept[n_pre:rest][never].any(), f"{what}: a unit below the band was kept"
    exact = np.array_equal(np.flatnonzero(kept), np.asarray(oracle_keep))
    if tau_hi - tau_lo > BAND:
        assert exact, f"{what}: index set differs although the gap is {tau_hi - tau_lo:.3g}"
    return exact


def import_oracle_state(gpu, st, int4: bool):
    if int4:
        gpu.import_state_int4(st["Kc"], st["Ks"], st["Vc"], st["Vs"], st["S"], st["T"], st["seen"])
    else:
        gpu.import_state(st["K"], st["V"], st["S"], st["T"], st["seen"])


def lockstep_chunk(ora, gpu, x: np.ndarray, flags: int = 0, rows=None, what=""):
    """Import the oracle's state, run one chunk on both, compare everything.  Advances the oracle."""
    shape = ora.s
    h, hk, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    n_tok = x.shape[0]
    st = ora.export_state()
    ln = ora.len
    xd = bf16_dev(x)
    out_a = torch.zeros((n_tok, h * d), dtype=torch.bfloat16, device="cuda")
    out_b = torch.zeros_like(out_a)

    # pass 1: append only, to read the chunk's K, V and scores before compaction
    int4 = bool(ora.int4)
    import_oracle_state(gpu, st, int4)
    gpu.prefill_chunk(xd, out_a, O.NO_EVICT)
    pre = gpu.export_state()
    assert gpu.sync_status() == 0
    # pass 2: the step as asked
    import_oracle_state(gpu, st, int4)
    gpu.prefill_chunk(xd, out_b, flags)
    post = gpu.export_state()
    assert gpu.sync_status() == 0
    assert torch.equal(out_a, out_b), f"{what}: attention output not reproducible"

    ref_out = ora.prefill_chunk(x, flags, rows=rows)
    stats = {}
    stats["attn_max_abs"] = check_attention(out_b.float().cpu().numpy().astype(np.float64), ref_out, what,
                                            ora.last_abs_out, ora.last_flip_sens)

    n = ln + n_tok
    assert pre["K"].shape[1] == n and pre["seen"] == st["seen"] + n_tok
    # imported part untouched, token ids appended
    assert np.array_equal(pre["K"][:, :ln], st["K"].astype(np.float32))
    state_keys = ("Kc", "Vc", "Ks", "Vs") if int4 else ("K", "V")
    assert np.array_equal(pre["T"][:, ln:], np.broadcast_to(st["seen"] + np.arange(n_tok), (hk, n_tok)))
    # chunk K, V as stored (bf16 of fp32 accumulation vs bf16 of fp64: rare one-ulp flips allowed)
    qkv = O.round_bf16(O.project_qkv(x, ora.w_qkv, h, hk, d))
    _, Kc, Vc = O.split_qkv(qkv, h, hk, d)
    if int4:
        # the chunk's units are stored quantised; a one-ulp difference in a staged bf16 value can
        # move a code by one step (or the scale by one fp16 ulp when it hits the absmax element)
        for name, src in (("K", Kc), ("V", Vc)):
            codes, scale = O.quantize_int4(np.transpose(src, (1, 0, 2)))
            got_c, got_s = pre[name + "c"][:, ln:], pre[name + "s"][:, ln:]
            assert np.array_equal(pre[name + "c"][:, :ln], st[name + "c"]), f"{what}: imported {name} codes changed"
            assert np.array_equal(pre[name + "s"][:, :ln], st[name + "s"].astype(np.float32))
            assert np.mean(got_s != scale.astype(np.float32)) < 0.01, f"{what}: {name} scales differ"
            assert np.mean(got_c != codes) < 0.01, f"{what}: {name} codes differ"
            deq_err = np.abs(got_c * got_s[..., None] - codes * scale[..., None])
            assert np.all(deq_err <= 1.001 * np.maximum(got_s, scale)[..., None]), f"{what}: {name} off by more than a step"
    for name, got, ref in (() if int4 else (("K", pre["K"][:, ln:], np.transpose(Kc, (1, 0, 2))),
                                            ("V", pre["V"][:, ln:], np.transpose(Vc, (1, 0, 2))))):
        diff = np.abs(got - ref)
        # one bf16 ulp of the value, plus the absolute error of an fp32 accumulation (matters
        # only for results that cancel to nearly zero)
        assert np.all(diff <= np.abs(ref) * 2.0 ** -7 + 1e-5 * np.abs(ref).max()), \
            f"{what}: chunk {name} off by more than one bf16 ulp"
        flips = float(np.mean(diff != 0))
        assert flips < FLIP_FRACTION, f"{what}: too many rounding flips in chunk {name}: {flips:.4f}"
    stats["score_worst"] = check_scores(pre["S"][:, ln:].T.astype(np.float64), ora.last_scores, what)

    evict = not (flags & O.NO_EVICT) and n > ora.budget
    if evict:
        n_prot = 0 if (flags & O.LAST_CHUNK) else min(ora.n_stab, n)
        s_ref = np.concatenate([st["S"], ora.last_scores.T], axis=1)
        exact = True
        for m in range(hk):
            pos = np.searchsorted(pre["T"][m], post["T"][m])
            assert np.array_equal(pre["T"][m][pos], post["T"][m]), f"{what}: unknown token id after compaction"
            assert np.all(np.diff(pos) > 0), f"{what}: temporal order lost"
            exact &= check_keep_band(pos, s_ref[m], ora.budget, n_prot, ora.last_keep[m], f"{what} head {m}", n_pre=ora.n_prefix)
            # compaction is a bit-exact gather of the pre-compaction arrays
            for key in state_keys:
                assert np.array_equal(post[key][m], pre[key][m][pos]), f"{what}: {key} not a bit-exact gather"
            assert np.array_equal(post["S"][m].view(np.uint32), pre["S"][m][pos].view(np.uint32))
        stats["sets_identical"] = exact
    else:
        for key in state_keys + ("T",):
            assert np.array_equal(post[key], pre[key])
    assert gpu.cache_len == ora.len
    return stats
