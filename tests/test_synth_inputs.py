"""The seeded input generators: any slice of any stream is reproducible on its own, the rows have the
shape the recipe states, and the manifold recipe really has the low intrinsic dimension it is there
for (input generation only: none of the method's arithmetic lives in that module)."""
import numpy as np
import pytest

from paper_2608_21163_b200 import synth


@pytest.mark.parametrize("name", sorted(synth.CONFIGS))
def test_any_slice_is_reproducible_on_its_own(name):
    cfg = synth.scaled(synth.CONFIGS[name], 0.001)
    wl = synth.Workload(cfg, seed=3)
    whole = wl.vectors(0, 300)
    part = wl.vectors(117, 50)
    assert whole.shape == (300, cfg["dim"]) and whole.dtype == (np.float32 if cfg["dtype"] == synth.F32 else np.uint8)
    assert (whole[117:167] == part).all()
    assert (wl.vectors(0, 300) == whole).all()
    other = synth.Workload(cfg, seed=4).vectors(0, 300)
    assert (other != whole).any()
    q = wl.queries()
    assert q.shape == (cfg["nq"], cfg["dim"]) and (q[: min(len(q), 300)] != whole[: min(len(q), 300)]).any()


def participation_ratio(x):
    """(sum of covariance eigenvalues)^2 / sum of their squares: the number of directions that carry the variance."""
    w = np.linalg.eigvalsh(np.cov(x.astype(np.float64).T))
    return w.sum() ** 2 / (w ** 2).sum()


def test_manifold_rows_are_unit_length_and_low_dimensional():
    x = synth.manifold_unit_f32(0, "base", 0, 6000, 96, latent=32, spread=1.0, noise=0.5)
    assert np.allclose(np.linalg.norm(x.astype(np.float64), axis=1), 1.0, atol=1e-6)
    iso = synth.gaussian_unit_f32(0, "base", 0, 6000, 96)
    pr_m, pr_i = participation_ratio(x), participation_ratio(iso)
    assert pr_m < 45 and pr_i > 85          # about the latent dimension against about the coordinate count
    # nearest neighbours stand out from the bulk on the manifold rows and hardly at all on isotropic ones
    def contrast(a):
        d = ((a[:100, None, :].astype(np.float64) - a[None, 100:3100, :]) ** 2).sum(-1)
        d.sort(1)
        return (d[:, 0] / np.median(d, 1)).mean()
    assert contrast(x) < 0.5 < contrast(iso)


def test_gist_shaped_rows_are_non_negative():
    x = synth.manifold_abs_f32(1, "base", 0, 500, 960)
    assert x.dtype == np.float32 and (x >= 0).all() and x.max() < 10.0


def test_isotropic_stress_config_keeps_the_deep_shaped_sizes():
    a, b = synth.CONFIGS["deep_f32_d96"], synth.CONFIGS["deep_f32_d96_isotropic"]
    for k in ("dim", "dtype", "metric", "mode", "R", "L", "alpha", "n", "build", "ins", "dele", "nq"):
        assert a[k] == b[k]
    assert a["gen"] != b["gen"]
