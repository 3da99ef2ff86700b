"""The harness metrics against closed forms (no GPU): PSNR from a known error, SSIM of identical
and of constant images, and monotonic behaviour under noise; the procedural target is seeded."""
import math

import numpy as np

import dhq_inputs
from paper_2508_13478_b200 import quality


def test_psnr_of_a_known_error():
    a = np.zeros((8, 8, 1))
    assert quality.psnr(a, a) == float("inf")
    assert math.isclose(quality.psnr(a, a + 0.1), 20.0, rel_tol=1e-12)          # mse 0.01 -> 20 dB
    assert math.isclose(quality.psnr(a, a + 0.01, peak=1.0), 40.0, rel_tol=1e-12)


def test_ssim_closed_forms_and_monotonicity():
    rng = np.random.default_rng(0)
    img = dhq_inputs.procedural_image(64, 64, 1, 3)
    assert math.isclose(quality.ssim(img, img), 1.0, rel_tol=1e-12)
    # two constant images c1, c2: variances and covariance vanish, SSIM = (2 c1 c2 + C1) / (c1^2 + c2^2 + C1)
    c1, c2 = 0.3, 0.5
    a, b = np.full((32, 32, 1), c1), np.full((32, 32, 1), c2)
    assert math.isclose(quality.ssim(a, b), (2 * c1 * c2 + 1e-4) / (c1 * c1 + c2 * c2 + 1e-4), rel_tol=1e-9)
    s1 = quality.ssim(img, np.clip(img + rng.normal(0, 0.02, img.shape), 0, 1))
    s2 = quality.ssim(img, np.clip(img + rng.normal(0, 0.1, img.shape), 0, 1))
    assert 1.0 > s1 > s2 > 0.0


def test_procedural_image_is_seeded_and_has_structure():
    a = dhq_inputs.procedural_image(64, 48, 3, 5)
    b = dhq_inputs.procedural_image(64, 48, 3, 5)
    c = dhq_inputs.procedural_image(64, 48, 3, 6)
    assert a.shape == (64, 48, 3) and a.dtype == np.float32 and np.array_equal(a, b) and not np.array_equal(a, c)
    assert a.min() >= 0.0 and a.max() <= 1.0 and a.std() > 0.05
    assert np.abs(np.diff(a[:, :, 0], axis=1)).max() > 0.1                        # hard edges are there
