"""The one rule every GPU test applies to the projected gradient g of Eq. (1) (helper, not a test module).

g = (L+ - L-) / (2 eps) amplifies a loss difference by 500 at eps = 1e-3 and the quantised forward is
discontinuous, so two correct implementations differ by far more than 2e-3 relative on most steps: the float64
oracle disagrees with its own run under binary32 storage of activations (OracleConfig.store_f32) by about 1-2 % of
rms(g) on the multi-layer configurations.  That self-disagreement ("band") is measured on the same inputs, step by
step.  It models only part of what a binary32 implementation does differently (storage, not accumulation order or
the binary16 attention operands) and collapses to 0.03 % of rms(g) on the smallest models while the GPU's distance
stays near 0.3 %, so the rms bound never drops below 1 % of rms(g).

records: dicts with g (float64 oracle), g32 (the oracle under binary32 storage, same weights) and g_gpu, one per
evaluated direction, every step state-synced (GPU masters copied from the oracle before it).
"""
import numpy as np


def check_g(recs, label):
    g = np.array([r["g"] for r in recs]); g32 = np.array([r["g32"] for r in recs]); gg = np.array([r["g_gpu"] for r in recs])
    g_rms = float(np.sqrt(np.mean(g * g)))
    band_rms = float(np.sqrt(np.mean((g - g32) ** 2)))
    err = np.abs(gg - g)
    err_rms = float(np.sqrt(np.mean(err ** 2)))
    err32_rms = float(np.sqrt(np.mean((gg - g32) ** 2)))
    target = 2e-3 * np.maximum(np.abs(g), g_rms)
    within_target = int(np.sum(err <= target))
    band_within = int(np.sum(np.abs(g - g32) <= target))
    # the line the measured table of the design notes is made of
    print(f"[g parity {label}] n {len(recs)}; rms g {g_rms:.4f}; rms |g_gpu-g_oracle| {err_rms:.2e} ({err_rms / g_rms:.2%}); "
          f"oracle self-band rms {band_rms:.2e} ({band_rms / g_rms:.2%}); rms |g_gpu-g_oracle(store_f32)| {err32_rms:.2e} "
          f"({err32_rms / g_rms:.2%}); steps within 2e-3: {within_target}/{len(recs)} "
          f"(the oracle against its own store_f32 run: {band_within}/{len(recs)})")
    assert err_rms <= max(3.0 * band_rms, 1e-2 * g_rms) + 2e-3 * g_rms, (label, err_rms, band_rms, g_rms)
    assert np.all(err <= 0.05 * g_rms + 2e-3 * np.abs(g)), (label, float(err.max()), g_rms)
    if len(recs) >= 8:
        assert np.corrcoef(g, gg)[0, 1] > 0.995, label
