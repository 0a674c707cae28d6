"""The oracle against its pins (CPU only), and the pins against deliberately broken oracles."""
import os
import subprocess
import sys
import tempfile

import pytest

import oracle
from oracle_pins import ALL_PINS

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(os.path.dirname(HERE), "oracle", "oracle.c")


@pytest.mark.parametrize("pin", ALL_PINS, ids=lambda f: f.__name__)
def test_oracle_meets_pin(pin):
    pin(oracle.lib())


# (label, text in oracle.c, replacement): each is a plausible slip in one place of the oracle.
MUTANTS = [
    ("no_rounding_term", "int64_t r = (shift >= 1) ? ((int64_t)1 << (shift - 1)) : 0;", "int64_t r = 0;"),
    ("truncate_not_floor", "if (rem < 0) q -= 1;", ""),
    ("relu_dropped", "if (relu && t < 0) t = 0;", ""),
    ("clamp_hi_128", "if (u > 127) u = 127;", "if (u > 128) u = 128;"),
    ("clamp_lo_127", "if (u < -128) u = -128;", "if (u < -127) u = -127;"),
    ("bias_subtracted", "int64_t t = acc + (int64_t)bias;", "int64_t t = acc - (int64_t)bias;"),
    ("round_term_full", "((int64_t)1 << (shift - 1))", "((int64_t)1 << shift)"),
    ("gemm_b_strides_swapped",
     "acc += (int32_t)A[m * a_rs + k * a_cs] * (int32_t)B[k * b_rs + n * b_cs];\n            int ovf = 0;\n            C[m * ldc + n]",
     "acc += (int32_t)A[m * a_rs + k * a_cs] * (int32_t)B[n * b_rs + k * b_cs];\n            int ovf = 0;\n            C[m * ldc + n]"),
    ("gemm_acc_a_strides_swapped",
     "acc += (int32_t)A[m * a_rs + k * a_cs] * (int32_t)B[k * b_rs + n * b_cs];\n            ACC[",
     "acc += (int32_t)A[k * a_rs + m * a_cs] * (int32_t)B[k * b_rs + n * b_cs];\n            ACC["),
    ("gemm_channel_index_m", "mult[per_channel ? n : 0],\n                                                    shift[per_channel ? n : 0], &ovf);\n            overflow |= ovf;\n        }\n    return overflow;\n}\n\n/* batch",
     "mult[per_channel ? m : 0],\n                                                    shift[per_channel ? n : 0], &ovf);\n            overflow |= ovf;\n        }\n    return overflow;\n}\n\n/* batch"),
    ("batched_bias_stride_ignored", "bias ? bias + b * bias_bs : NULL", "bias ? bias : NULL"),
    ("batched_b_not_advanced", "const int8_t *Bb = B + b * b_bs;", "const int8_t *Bb = B;"),
    ("conv_kernel_flipped", "int h = p * stride_h - pad_h + r;", "int h = p * stride_h - pad_h + (R - 1 - r);"),
    ("conv_pad_sign", "int ww = q * stride_w - pad_w + s;", "int ww = q * stride_w + pad_w + s;"),
    ("conv_stride_ignored_w", "int ww = q * stride_w - pad_w + s;", "int ww = q - pad_w + s;"),
    ("conv_h_w_swapped", "((int64_t)n * H + h) * W + ww) * C", "((int64_t)n * H + ww) * W + h) * C"),
    ("conv_extent_ceil", "int Q = (W + 2 * pad_w - S) / stride_w + 1;", "int Q = (W + 2 * pad_w - S + stride_w - 1) / stride_w + 1;"),
    ("conv_bound_off_by_one", "if (h < 0 || h >= H) continue;", "if (h < 0 || h >= H - 1) continue;"),
    ("fscale_truncates", "return (int32_t)lrintf(y);", "return (int32_t)y;"),
    ("fscale_ties_away", "return (int32_t)lrintf(y);", "return (int32_t)roundf(y);"),
    ("fscale_double_product", "volatile float y = tf * scale;", "volatile float y = (float)((double)(int32_t)t * (double)scale);"),
    ("fscale_relu_after_scale", "if (relu && t < 0) t = 0;\n    volatile float tf", "volatile float tf"),
    ("fscale_bias_dropped", "int64_t t = acc + (int64_t)bias;\n    if (overflow && (t > (int64_t)INT32_MAX || t < (int64_t)INT32_MIN)) *overflow = 1;\n    if (relu && t < 0) t = 0;\n    volatile float tf",
     "int64_t t = acc;\n    if (relu && t < 0) t = 0;\n    volatile float tf"),
    ("fscale_clamp_hi_128", "if (y >= 127.0f) return 127;", "if (y >= 128.0f) return 128;"),
    ("fscale_channel_index_m", "scale[per_channel ? n : 0], &ovf);", "scale[per_channel ? m : 0], &ovf);"),
    ("conv_weight_layout_kcrs", "(((int64_t)k * R + r) * S + s) * C", "(((int64_t)k * S + s) * R + r) * C"),
]


@pytest.mark.parametrize("label,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_pins_catch_planted_mistake(label, old, new):
    """A mistake planted in a copy of the oracle (on the CPU) must fail at least one pin."""
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation site for {label} not found"
    with tempfile.TemporaryDirectory() as d:
        src = os.path.join(d, "oracle_mut.c")
        so = os.path.join(d, "liboracle_mut.so")
        open(src, "w").write(text.replace(old, new, 1))
        subprocess.run(["gcc", "-O1", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", so, src, "-lm"], check=True)
        # The pins run in a child process: a planted indexing mistake may write outside the oracle's buffers, and a
        # crash of the child counts as "noticed" just like a failed assertion.
        code = ("import sys; sys.path.insert(0, %r); sys.path.insert(0, %r)\n"
                "import oracle\nfrom oracle_pins import ALL_PINS\n"
                "m = oracle.Oracle(%r)\n"
                "for pin in ALL_PINS:\n"
                "    try:\n        pin(m)\n"
                "    except Exception:\n        sys.exit(3)\n"
                "sys.exit(0)\n") % (os.path.dirname(HERE), HERE, so)
        rc = subprocess.run([sys.executable, "-c", code], capture_output=True).returncode
        caught = rc != 0
        assert caught, f"no pin noticed the planted mistake '{label}'"
