"""Do the pins bite?  Each case plants ONE plausible mistake in a copy of the C oracle (a wrong
sign, a dropped factor, another rounding, a transposed operand, a dropped term), compiles that
copy on the CPU, lets the oracle's Python driver load it in place of the real library and runs the
pin tests against it: at least one pin must fail.  The unmodified source, taken through the same
machinery, must pass all of them.  Nothing here touches a GPU or the CUDA library.
"""
import os
import subprocess

import pytest

from oracle import dhq_oracle as orc
from tests import test_oracle_pins as pins
from tests import test_oracle_tiers as tiers
from tests.conftest import load_golden

SRC = os.path.join(os.path.dirname(os.path.abspath(orc.__file__)), "dhq_oracle.c")

# (name, text in dhq_oracle.c that occurs exactly once, its replacement)
MUTATIONS = [
    ("hadamard_lower_right_block_not_negated",
     "H[(size_t)(i + m) * n + (j + m)] = (int8_t)(-h);", "H[(size_t)(i + m) * n + (j + m)] = h;"),
    ("hadamard_lower_left_block_negated",
     "H[(size_t)(i + m) * n + j] = h;", "H[(size_t)(i + m) * n + j] = (int8_t)(-h);"),
    ("rotation_sign_of_products_flipped",
     "scratch[l] = (row[l] > 0) ? v[l] : -v[l];", "scratch[l] = (row[l] > 0) ? -v[l] : v[l];"),
    ("rotation_summed_left_to_right",
     "    float a = pairwise_sum_f32(t, lo, len / 2);\n    float b = pairwise_sum_f32(t, lo + len / 2, len / 2);\n    return a + b;",
     "    float a = t[lo];\n    for (int i = 1; i < len; ++i) a += t[lo + i];\n    return a;"),
    ("qmax_is_two_to_the_b_minus_one_in_the_scales",
     "float qmax = (float)((1 << (bits - 1)) - 1);", "float qmax = (float)(1 << (bits - 1));"),
    ("qmax_is_two_to_the_b_minus_one_in_the_clamp",
     "int32_t qmax = (1 << (bits - 1)) - 1;", "int32_t qmax = (1 << (bits - 1));"),
    ("round_half_away_from_zero", "float r = rintf(t);", "float r = roundf(t);"),
    ("truncation_instead_of_rounding", "float r = rintf(t);", "float r = truncf(t);"),
    ("no_upper_clamp", "if (r > (float)qmax) r = (float)qmax;", ""),
    ("scale_is_the_absmax_itself", "*s = a / qmax;", "*s = a;"),
    ("weight_fold_without_one_over_k", "float invK = 1.0f / (float)K_pad;", "float invK = 1.0f;"),
    ("weights_padded_transposed",
     "padded[(size_t)m * K_pad + k] = W[(size_t)m * d_in + k];", "padded[(size_t)m * K_pad + k] = W[(size_t)k * d_out + m];"),
    ("per_channel_rows_share_the_first_rows_scale",
     "dhq_orc_scales(dhq_orc_absmax(Wrot + (size_t)m * K_pad, K_pad), bits, &s, &inv);",
     "dhq_orc_scales(dhq_orc_absmax(Wrot, K_pad), bits, &s, &inv);"),
    ("two_sided_without_one_over_m", "float invM = 1.0f / (float)M_pad;", "float invM = 1.0f;"),
    ("activations_not_rotated",
     "            if (rotate) rotate_one(H, K_pad, x, xr, scratch);\n            else memcpy(xr, x, sizeof(float) * (size_t)K_pad);\n            float a = per_token",
     "            memcpy(xr, x, sizeof(float) * (size_t)K_pad);\n            float a = per_token"),
    ("matmul_reads_the_weights_of_the_wrong_row",
     "const int32_t *wr = qw + (size_t)m * K_pad;", "const int32_t *wr = qw + (size_t)(M_pad - 1 - m) * K_pad;"),
    ("bias_dropped",
     "double z = (double)s_w[m] * (double)s * (double)sum + (double)b_pad[m];", "double z = (double)s_w[m] * (double)s * (double)sum;"),
    ("activation_scale_left_out_of_the_dequantization",
     "double z = (double)s_w[m] * (double)s * (double)sum + (double)b_pad[m];", "double z = (double)s_w[m] * (double)sum + (double)b_pad[m];"),
    ("omega0_left_out", "double y = sin(omega0 * z);", "double y = sin(z);"),
    ("cosine_instead_of_sine", "double y = sin(omega0 * z);", "double y = cos(omega0 * z);"),
    ("last_layer_gets_the_activation",
     "Y[t * M_pad + m] = apply_sine ? activation(z, omega0, gabor_s0) : z;", "Y[t * M_pad + m] = activation(z, omega0, gabor_s0);"),
    ("two_sided_output_not_rotated_back",
     "for (int m = 0; m < M_pad; ++m) z += (hr[m] > 0) ? dq[m] : -dq[m];", "z = dq[j];"),
    ("gabor_envelope_without_the_square",
     "y *= exp(-(gabor_s0 * z) * (gabor_s0 * z));", "y *= exp(-fabs(gabor_s0 * z));"),
    ("per_token_absmax_ignored_for_the_frozen_value",
     "float a = per_token ? dhq_orc_absmax(xr, K_pad) : a_frozen;", "float a = per_token ? dhq_orc_absmax(x, K_pad) : a_frozen;"),
]


def _battery():
    """The pins run against every mutant, cheap ones first (a mutant stops at its first failure)."""
    g = load_golden
    return [
        ("hadamard", lambda: pins.test_hadamard_recursion_equals_closed_form_and_is_orthogonal(8)),
        ("h4 rows", pins.test_hadamard_h4_rows_as_printed_by_the_recursion),
        ("rotation on integers", lambda: pins.test_rotation_exact_on_small_integers(8)),
        ("rotation against fp64", lambda: pins.test_rotation_close_to_fp64_product(64)),
        ("fixture F1 (rotation)", lambda: pins.test_rotation_fixture_f1(g)),
        ("fixture F4 (summation order)", lambda: pins.test_rotation_summation_order_fixture_f4(g)),
        ("butterfly form", lambda: pins.test_butterfly_form_is_bit_identical_to_the_tree_definition(32)),
        ("quantizer properties, 4 bits", lambda: pins.test_quantizer_properties(4)),
        ("quantizer properties, 8 bits", lambda: pins.test_quantizer_properties(8)),
        ("fixtures F1, F2 (quantizer)", lambda: pins.test_quantizer_fixtures_f1_f2(g)),
        ("zero input and saturation", pins.test_quantizer_zero_input_and_saturation),
        ("weight fold", lambda: pins.test_weight_fold_norm_and_compute_invariance((64, 64))),
        ("weight fold, first layer", lambda: pins.test_weight_fold_norm_and_compute_invariance((64, 2))),
        ("fixture F3 (weight fold)", lambda: pins.test_weight_fold_fixture_f3(g)),
        ("fixture F5 (per-channel scales)", lambda: tiers.test_per_channel_weight_quantizer_fixture_f5(g)),
        ("brute force, 2 bits", lambda: pins.test_brute_force_all_code_vectors_on_a_4_wide_layer(2)),
        ("integer matmul and sine", pins.test_integer_matmul_matches_int64_product_and_hidden_layers_apply_sine),
        ("padding of first and last layer", pins.test_first_layer_pads_coordinates_and_last_layer_pads_outputs),
        ("zero token", pins.test_zero_token_has_zero_codes_per_token),
        ("two-sided weights", lambda: pins.test_two_sided_weight_transform_matches_eq5_and_keeps_the_product((64, 64))),
        ("two-sided layer, exact rationals", pins.test_two_sided_layer_brute_force_with_exact_rationals),
        ("wavelet by hand", tiers.test_gabor_activation_by_hand_and_its_limits),
        ("two tiers", lambda: tiers.test_fp32_oracle_codes_agree_with_the_fp64_orthonormal_statement("C1", 4096, 0, 0)),
        ("convergence", pins.test_quantized_network_converges_to_the_unquantized_siren),
    ]


def _compile(text, path):
    src = path + ".c"
    with open(src, "w") as f:
        f.write(text)
    subprocess.run(["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared",
                    "-fvisibility=hidden", "-o", path, src, "-lm"], check=True)
    return path


@pytest.fixture()
def swap_oracle_library(monkeypatch):
    """Lets the oracle's driver load another build of its C file; the real one comes back afterwards."""
    def swap(path):
        monkeypatch.setattr(orc, "build", lambda force=False: path)
        monkeypatch.setattr(orc, "_lib", None)
    yield swap
    monkeypatch.undo()
    orc._lib = None


def _first_failure():
    for name, pin in _battery():
        try:
            pin()
        except (AssertionError, ValueError, FloatingPointError, ZeroDivisionError) as e:
            return name, e
    return None, None


def test_the_unmodified_source_passes_the_battery(tmp_path, swap_oracle_library):
    swap_oracle_library(_compile(open(SRC).read(), str(tmp_path / "liborc_control.so")))
    name, err = _first_failure()
    assert name is None, f"control build failed pin '{name}': {err}"


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_a_planted_mistake_fails_a_pin(name, old, new, tmp_path, swap_oracle_library):
    text = open(SRC).read()
    assert text.count(old) == 1, "the text to mutate must occur exactly once in dhq_oracle.c"
    swap_oracle_library(_compile(text.replace(old, new), str(tmp_path / f"liborc_{name}.so")))
    pin, err = _first_failure()
    assert pin is not None, f"no pin noticed the planted mistake '{name}'"
    print(f"{name}: caught by '{pin}'")


# The oracle's Python driver (padding, chaining, calibration) gets the same treatment: one function
# at a time is re-created from its source text with one mistake and put in the module's place.
DRIVER_MUTATIONS = [
    ("coordinates_padded_into_the_wrong_slots", "pad_coords", "X[:, : c.shape[1]] = c", "X[:, 4 - c.shape[1]:] = c"),
    ("bias_padded_at_the_wrong_end", "prepare", "b_pad[:d_out] = _f32(biases[l - 1])", "b_pad[M_pad - d_out:] = _f32(biases[l - 1])"),
    ("last_layer_marked_as_a_sine_layer", "prepare", "sine=(l < L)", "sine=True"),
    ("padded_sizes_of_the_last_layer_not_applied", "pad_dims", "M_pad = 4 if l == L else int(dims[l])", "M_pad = 4 if l == 1 else int(dims[l])"),
    ("calibration_takes_the_mean", "calibrate", "rotated_absmax(net, l, X).max()", "rotated_absmax(net, l, X).mean()"),
    ("calibration_does_not_advance_through_the_layers", "calibrate",
     'X = layer(net, l, X, want=("Y",))["Y"].astype(np.float32)', "X = np.zeros((X.shape[0], net.layers[l].K_pad), np.float32) + X[:, :1]"),
    ("granularity_flag_inverted", "layer", "per_token = int(net.a_gran == 1)", "per_token = int(net.a_gran == 0)"),
    ("forward_returns_the_wrong_output_columns", "forward", 'out = r["Y"][:, : net.dims[-1]]', 'out = r["Y"][:, -net.dims[-1]:]'),
    ("chain_not_rounded_to_fp32_inputs_but_restarted", "forward", 'X = r["Y"].astype(np.float32)', 'X = np.abs(r["Y"]).astype(np.float32)'),
]


def _driver_battery():
    return [
        ("padding of first and last layer", pins.test_first_layer_pads_coordinates_and_last_layer_pads_outputs),
        ("brute force, 2 bits", lambda: pins.test_brute_force_all_code_vectors_on_a_4_wide_layer(2)),
        ("integer matmul and sine", pins.test_integer_matmul_matches_int64_product_and_hidden_layers_apply_sine),
        ("calibration", pins.test_per_tensor_calibration_is_the_layerwise_maximum_and_freezes),
        ("zero token", pins.test_zero_token_has_zero_codes_per_token),
        ("two tiers", lambda: tiers.test_fp32_oracle_codes_agree_with_the_fp64_orthonormal_statement("C1", 4096, 0, 0)),
        ("convergence", pins.test_quantized_network_converges_to_the_unquantized_siren),
    ]


@pytest.mark.parametrize("name,fn_name,old,new", DRIVER_MUTATIONS, ids=[m[0] for m in DRIVER_MUTATIONS])
def test_a_planted_mistake_in_the_driver_fails_a_pin(name, fn_name, old, new, monkeypatch):
    import inspect
    src = inspect.getsource(getattr(orc, fn_name))
    assert src.count(old) == 1, "the text to mutate must occur exactly once in the function"
    made = {}
    exec(compile(src.replace(old, new), f"<{fn_name} with a planted mistake>", "exec"), orc.__dict__, made)
    monkeypatch.setattr(orc, fn_name, made[fn_name])
    caught = None
    for pin_name, pin in _driver_battery():
        try:
            pin()
        except (AssertionError, ValueError, IndexError, RuntimeError, OverflowError):
            caught = pin_name
            break
    assert caught is not None, f"no pin noticed the planted mistake '{name}'"
    print(f"{name}: caught by '{caught}'")
