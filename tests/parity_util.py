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
WELL_CONDITIONED = 5e-3  # an output element is well conditioned when the oracle's own first-order estimate of what
                         # the legitimate storage differences can do to it, (P_ULP + V_ULP) sum p|v| + flip_sens,
                         # stays below this: the row puts no weight worth mentioning on a 20x-norm outlier
                         # token.  There the stated tolerance (max-abs 2e-2) is asserted as it is written.


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


def attention_stats(got: np.ndarray, ref: np.ndarray, abs_ref=None, flip_sens=None, pure_ref=None, head_dim=None):
    """How much of the derived bound the comparison uses, and how the CUDA path fares against the
    plain stated tolerance (max-abs 2e-2), per chunk:
      plain_max_abs            largest |delta| over all compared elements
      plain_exceed_share       share of elements beyond the plain mixed bound 2e-2 * max(1, |ref|)
                               (these are the ones that need the derived terms)
      wellcond_share / wellcond_max_abs   share of elements whose derived terms stay below WELL_CONDITIONED
                               (no weight on an outlier token), and the largest |delta| on them (must stay
                               within the plain 2e-2)
      bound_used_max           worst err / full bound
      pure_within_2e-2_share   share of elements within plain 2e-2 of the oracle WITHOUT bf16 mirroring
    """
    rows = ~np.isnan(ref).any(axis=1)
    g, r = got[rows], ref[rows]
    err = np.abs(g - r)
    st = {"plain_max_abs": float(err.max()) if err.size else 0.0,
          "plain_exceed_share": float(np.mean(err > ATTN_TOL * np.maximum(1.0, np.abs(r)))) if err.size else 0.0}
    if abs_ref is not None:
        bound = ATTN_TOL * np.maximum(1.0, np.abs(r)) + (P_ULP + V_ULP) * abs_ref[rows]
        if flip_sens is not None:
            bound = bound + flip_sens[rows]
        st["bound_used_max"] = float(np.max(err / bound)) if err.size else 0.0
        extra = bound - ATTN_TOL * np.maximum(1.0, np.abs(r))
        well = extra <= WELL_CONDITIONED
        st["rows"] = int(rows.sum())
        st["wellcond_share"] = float(np.mean(well)) if well.size else 0.0
        st["wellcond_max_abs"] = float(err[well].max()) if well.any() else 0.0
    if pure_ref is not None:
        st["pure_within_2e-2_share"] = float(np.mean(np.abs(g - pure_ref[rows]) <= ATTN_TOL))
        st["pure_max_abs"] = float(np.max(np.abs(g - pure_ref[rows])))
    return st


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


def lockstep_chunk(ora, gpu, x: np.ndarray, flags: int = 0, rows=None, what="", pure=None, plain=False):
    """Import the oracle's state, run one chunk on both, compare everything.  Advances the oracle.
    pure: an OracleLayer with mirror=False that is given the same state and chunk; its output only
    feeds the statistics (how the CUDA path fares against the un-mirrored fp64 result).
    plain: also assert the plain stated tolerances (attention max-abs 2e-2; workloads without
    outlier tokens)."""
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

    pure_out = None
    if pure is not None:
        pure.import_state(st)
        pure_out = pure.prefill_chunk(x, flags, rows=rows)
    ref_out = ora.prefill_chunk(x, flags, rows=rows)
    stats = {}
    got_out = out_b.float().cpu().numpy().astype(np.float64)
    stats["attn_max_abs"] = check_attention(got_out, ref_out, what, ora.last_abs_out, ora.last_flip_sens)
    stats.update(attention_stats(got_out, ref_out, ora.last_abs_out, ora.last_flip_sens, pure_out, head_dim=d))
    # elements that put no weight on an outlier token meet the stated tolerance as it is written
    assert stats["wellcond_max_abs"] <= ATTN_TOL, \
        f"{what}: well-conditioned elements off by {stats['wellcond_max_abs']:.4g} (plain tolerance {ATTN_TOL})"
    if plain:
        assert stats["plain_max_abs"] <= ATTN_TOL, f"{what}: plain max-abs {stats['plain_max_abs']:.4g}"

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
        stats[f"flip_rate_{name}"] = flips
    got_s = pre["S"][:, ln:].T.astype(np.float64)
    stats["score_worst"] = check_scores(got_s, ora.last_scores, what)
    stats["score_plain_rel_worst"] = float(np.max(np.abs(got_s - ora.last_scores) /
                                                  np.maximum(np.abs(ora.last_scores), 1e-3)))

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


def forced_state(shape, budget: int, chunk: int, seed: int = 0, unmoved: int = 64):
    """A full cache whose next eviction is decided before any chunk score is known: budget - chunk
    units score +100 and chunk units score -100 (interleaved at random behind a short all-high
    prefix), so a full chunk with the last n_stab protected evicts exactly the -100 units whatever
    the chunk's own scores (|score| << 100): both sides keep the same set, the kept high units
    behind the prefix all move to new slots, and the prefix stays where it is."""
    import workloads as W
    hk, d = shape.n_kv_heads, shape.head_dim
    g = np.random.default_rng(7000 + seed)
    K = W.to_bf16_grid(g.standard_normal((hk, budget, d)).astype(np.float32)).astype(np.float64)
    V = W.to_bf16_grid(g.standard_normal((hk, budget, d)).astype(np.float32)).astype(np.float64)
    n_high = budget - chunk
    unmoved = min(unmoved, n_high)
    S = np.full((hk, budget), -100.0)
    for m in range(hk):
        S[m, :unmoved] = 100.0
        pick = unmoved + g.choice(budget - unmoved, size=n_high - unmoved, replace=False)
        S[m, pick] = 100.0
    T = np.broadcast_to(np.arange(budget, dtype=np.int64), (hk, budget)).copy()
    return dict(K=K, V=V, S=S, T=T, seen=budget)


def run_pair_without_reimport(ora, gpu, st, x_a, x_b, rows_a=None, rows_b=None, what=""):
    """Chunk A evicts and compacts from the forced state `st`; chunk B then runs on BOTH sides from
    what each side's own step A left (no import in between), so the attention of B reads the rotated
    keys that the CUDA compaction wrote.  Returns B's statistics."""
    h, d = ora.s.n_q_heads, ora.s.head_dim
    budget = ora.budget
    ora.import_state(st)
    gpu.import_state(st["K"], st["V"], st["S"], st["T"], st["seen"])
    out_a = torch.zeros((x_a.shape[0], h * d), dtype=torch.bfloat16, device="cuda")
    gpu.prefill_chunk(bf16_dev(x_a), out_a, 0)
    ref_a = ora.prefill_chunk(x_a, 0, rows=rows_a)
    check_attention(out_a.float().cpu().numpy().astype(np.float64), ref_a, f"{what} A", ora.last_abs_out,
                    ora.last_flip_sens)
    post = gpu.export_state()                       # reads the state; rotated keys are left as compaction wrote them
    assert gpu.sync_status() == 0
    assert np.array_equal(post["T"], ora.T), f"{what}: retained token ids differ after the forced eviction"
    keep = ora.last_keep
    moved = sum(int(np.sum(keep[m] != np.arange(budget))) for m in range(ora.hk))
    stay = sum(int(np.sum(keep[m] == np.arange(budget))) for m in range(ora.hk))
    assert moved > 0 and stay > 0, f"{what}: the forced eviction must both move and leave units"
    # the cache contents agree up to the rare one-ulp flips of the chunk's stored K, V
    for name in ("K", "V"):
        diff = np.abs(post[name] - getattr(ora, name))
        assert np.all(diff <= np.abs(getattr(ora, name)) * 2.0 ** -7 + 1e-5 * np.abs(getattr(ora, name)).max())
        assert np.mean(diff != 0) < FLIP_FRACTION
    out_b = torch.zeros((x_b.shape[0], h * d), dtype=torch.bfloat16, device="cuda")
    ln = ora.len
    gpu.prefill_chunk(bf16_dev(x_b), out_b, O.NO_EVICT)
    ref_b = ora.prefill_chunk(x_b, O.NO_EVICT, rows=rows_b)
    got_b = out_b.float().cpu().numpy().astype(np.float64)
    stats = {"attn_max_abs": check_attention(got_b, ref_b, f"{what} B", ora.last_abs_out, ora.last_flip_sens)}
    stats.update(attention_stats(got_b, ref_b, ora.last_abs_out, ora.last_flip_sens, head_dim=d))
    assert stats["wellcond_max_abs"] <= ATTN_TOL, f"{what} B: well-conditioned elements off by {stats['wellcond_max_abs']:.4g}"
    after = gpu.export_state()
    stats["score_worst"] = check_scores(after["S"][:, ln:].T.astype(np.float64), ora.last_scores, f"{what} B")
    stats["moved"], stats["stayed"] = moved, stay
    assert gpu.sync_status() == 0
    return stats
