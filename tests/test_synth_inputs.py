"""The seeded input generators both sides draw from (CPU only): what the configuration runs rely on."""
import numpy as np

from paper_2407_08296_b200 import synth


def test_column_block_sampler_is_consistent_and_has_the_planted_spectrum():
    gm = synth.GradientModel(300, 700, seed=1, matrix_index=2)
    full = gm.sample_columns(3, 0, 700)
    assert full.shape == (300, 700) and full.dtype == np.uint16
    for a, b in ((0, 256), (256, 512), (512, 700), (512, 600), (256, 700)):
        assert np.array_equal(full[:, a:b], gm.sample_columns(3, a, b))          # any range = its slice of the whole
    assert not np.array_equal(full, gm.sample_columns(4, 0, 700))                # fresh noise per step
    sv = np.linalg.svd(synth.bf16_bits_to_float(full).astype(np.float64), compute_uv=False)
    assert np.allclose(sv[:4], [1.0, 0.5, 1.0 / 3, 0.25], rtol=2e-2)             # planted 1/k above a 1e-3 noise floor
    assert sv[40] < 0.06


def test_rotation_turns_the_planted_subspace_by_the_stated_angle():
    gm = synth.GradientModel(256, 128, seed=3, matrix_index=0)
    U0 = gm.U.copy()
    gm.rotate(0.0, 1)
    assert np.allclose(np.abs(np.linalg.svd(U0.T @ gm.U, compute_uv=False)), 1.0)   # theta = 0: the same subspace
    theta = 0.7
    gm.rotate(theta, 2)
    assert np.allclose(gm.U.T @ gm.U, np.eye(gm.U.shape[1]), atol=1e-12)
    cosines = np.linalg.svd(U0.T @ gm.U, compute_uv=False)
    assert np.allclose(cosines, np.cos(theta), atol=1e-9)                            # every principal angle is theta
    gm.rotate(np.pi / 2, 3)
    U1 = gm.U.copy()
    gm2 = synth.GradientModel(256, 128, seed=3, matrix_index=0)
    gm2.rotate(0.0, 1); gm2.rotate(theta, 2); gm2.rotate(np.pi / 2, 3)
    assert np.array_equal(U1, gm2.U)                                                 # seeded: reproducible


def test_stack_shapes_and_seeds():
    assert len(synth.stack_matrices("llama130m")) == 84 and len(synth.stack_matrices("llama350m")) == 168
    assert len(synth.stack_matrices("llama1b")) == 168 and len(synth.stack_matrices("llama7b")) == 224
    assert synth.distinct_shapes("llama7b") == [(4096, 4096, 1024, 128), (4096, 11008, 1024, 64), (11008, 4096, 1024, 32)]
    assert synth.matrix_seed(3, 5) == (3 << 20) + 5
