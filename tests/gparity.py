"""The one rule every GPU test applies to the projected gradient g of Eq. (1) (helper, not a test module).

g = (L+ - L-) / (2 eps) amplifies a loss difference by 500 at eps = 1e-3 and the quantised forward is
discontinuous, so two correct implementations differ by far more than 2e-3 relative on most steps: the float64
oracle disagrees with its own runs in binary32 - activations merely stored in binary32 (OracleConfig.store_f32), or
every sum also accumulated in binary32 in the library's order (OracleConfig.accum_f32) - by up to a few per cent of
rms(g).  That self-disagreement ("band": the larger of the two, in rms over the steps) is measured on the same
inputs, step by step.  It is heavy-tailed (one differing code in one step dominates a short run) and models only part
of what another binary32 implementation does differently (not the tensor cores' accumulation order or the binary16
attention operands); on the small test models (a few hundred tokens) a single differing code moves g by 1-4 % of
rms(g), and whether a four-step run of the oracle's own binary32 variant catches one is luck, so the rms bound never
drops below 2.5 % of rms(g).

records: dicts with g (float64 oracle), g32 (the oracle under binary32 storage, same weights), optionally ga32 (the
oracle with binary32 accumulation) and g_gpu, one per evaluated direction, every step state-synced (GPU masters
copied from the oracle before it).
"""
import numpy as np


def check_g(recs, label):
    g = np.array([r["g"] for r in recs]); g32 = np.array([r["g32"] for r in recs]); gg = np.array([r["g_gpu"] for r in recs])
    g_rms = float(np.sqrt(np.mean(g * g)))
    band_store = float(np.sqrt(np.mean((g - g32) ** 2)))
    ga32 = np.array([r.get("ga32", r["g32"]) for r in recs])
    band_accum = float(np.sqrt(np.mean((g - ga32) ** 2)))
    band_rms = max(band_store, band_accum)
    err = np.abs(gg - g)
    err_rms = float(np.sqrt(np.mean(err ** 2)))
    err32_rms = float(np.sqrt(np.mean((gg - g32) ** 2)))
    target = 2e-3 * np.maximum(np.abs(g), g_rms)
    within_target = int(np.sum(err <= target))
    band_within = int(np.sum(np.abs(g - g32) <= target))
    # the line the measured table of the design notes is made of
    if all(r.get("ga32") is not None and r["g32"] == r["ga32"] for r in recs):
        label += " (store_f32 run skipped: both bands are the accum_f32 run)"
    print(f"[g parity {label}] n {len(recs)}; rms g {g_rms:.4f}; rms |g_gpu-g_oracle| {err_rms:.2e} ({err_rms / g_rms:.2%}); "
          f"oracle self-band rms: store_f32 {band_store:.2e} ({band_store / g_rms:.2%}), accum_f32 {band_accum:.2e} ({band_accum / g_rms:.2%}); "
          f"rms |g_gpu-g_oracle(store_f32)| {err32_rms:.2e} "
          f"({err32_rms / g_rms:.2%}); steps within 2e-3: {within_target}/{len(recs)} "
          f"(the oracle against its own store_f32 run: {band_within}/{len(recs)})")
    rms_bound = max(3.0 * band_rms, 2.5e-2 * g_rms) + 2e-3 * g_rms
    assert err_rms <= rms_bound, (label, err_rms, band_rms, g_rms)
    # single steps: heavy-tailed, so three times the rms bound
    assert np.all(err <= 3.0 * rms_bound + 2e-3 * np.abs(g)), (label, float(err.max()), g_rms, band_rms)
    if len(recs) >= 8:
        assert np.corrcoef(g, gg)[0, 1] > 0.995, label
