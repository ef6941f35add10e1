"""Do the pins notice a mistake?  Each case compiles a copy of the oracle source with ONE
planted error (wrong tie direction, dropped term, wrong offset, transposed grouping, ...)
and requires at least one pin to fail.  The mistakes are planted in the oracle, on the CPU."""
import os
import subprocess

import pytest

import oracle_pins as pins
from oracle import fb4_oracle as orc

SRC = os.path.join(os.path.dirname(orc.__file__), "fb4_oracle.c")

MUTANTS = {
    "round_ties_down": ("if (dj <= bestd) { bestd = dj; best = j; }", "if (dj < bestd) { bestd = dj; best = j; }"),
    "dialect_ties_to_highest": ("if (best < 0 || err < best_err)", "if (best < 0 || err <= best_err)"),
    "exponent_offset_2": ("return ldexp(fabs(x), 3 - e);", "return ldexp(fabs(x), 2 - e);"),
    "floor_log2_off_by_one": ("e = ex - 1;", "e = ex;"),
    "midpoint_dropped": ("+ 0.25;", "+ 0.0;"),
    "squared_error": ("err += fabs(mid - (double)F[d * 8 + nearest_index(F + d * 8, mid)]);",
                      "{ double q_ = mid - (double)F[d * 8 + nearest_index(F + d * 8, mid)]; err += q_ * q_; }"),
    "strided_groups": ("if (v[g * gs + i] > m) m = v[g * gs + i];", "if (v[g + i * G] > m) m = v[g + i * G];"),
    "one_group_missing": ("for (int g = 0; g < G; ++g) {\n      double mid", "for (int g = 1; g < G; ++g) {\n      double mid"),
    "bin_width_one": ("double b = floor(2.0 * v);", "double b = 2.0 * floor(v);"),
    "stage1_ignored": ("cand = stage1[bin_of(vmax)] & allowed;", "cand = allowed;"),
    "seda_mask_ignored": ("cand = stage1[bin_of(vmax)] & allowed;", "cand = stage1[bin_of(vmax)];"),
    "sign_dropped": ("code[i] = (uint8_t)((sgn[i] << 3) |", "code[i] = (uint8_t)((0 << 3) |"),
    "nibbles_swapped": ("(uint8_t)(code[i] | (code[i + 1] << 4));", "(uint8_t)(code[i + 1] | (code[i] << 4));"),
    "scale_byte_bias": ("(uint16_t)((e + 124) | (did << 8));", "(uint16_t)((e + 127) | (did << 8));"),
    "dequant_exponent": ("ldexp((double)F[did * 8 + (code & 7)], e - 3);", "ldexp((double)F[did * 8 + (code & 7)], e - 4);"),
    "residual_from_rounded_input": ("float df = (float)(xv[i] - dequant_value(F, did, e, code[i]));",
                                    "float df = (float)(xv[i] - 0.5 * dequant_value(F, did, e, code[i]));"),
    "residual_not_added": ("val = (float)((double)val + r);", "val = (float)((double)val + 0.0 * r);"),
    "salient_last_on_tie": ("if (score[t] > score[arg]) arg = t;", "if (score[t] >= score[arg]) arg = t;"),
    "salient_min": ("if (score[t] > score[arg]) arg = t;", "if (score[t] < score[arg]) arg = t;"),
    "topk_ties_to_highest": ("if (!taken[t] && (arg < 0 || score[t] > score[arg])) arg = t;",
                             "if (!taken[t] && (arg < 0 || score[t] >= score[arg])) arg = t;"),
    "topk_smallest": ("if (!taken[t] && (arg < 0 || score[t] > score[arg])) arg = t;",
                      "if (!taken[t] && (arg < 0 || score[t] < score[arg])) arg = t;"),
    "f16_through_bf16": ("_Float16 h = (_Float16)val;", "_Float16 h = (_Float16)bf16_to_double(f32_to_bf16_rne(val));"),
    "residual_ignores_seda_mask": ("quantize_block(dv, dsg, cfg, F, stage1, allowed, dcode, &rdid, &re, NULL);",
                                   "quantize_block(dv, dsg, cfg, F, stage1, 0xffffffffu, dcode, &rdid, &re, NULL);"),
    "clamp_min_ignored": ("if (e < cfg->exp_min) e = cfg->exp_min;", ";"),
    "zero_block_exponent": ("e = cfg->exp_min;\n  } else {", "e = 0;\n  } else {"),
    "stage1_bucket_shift": ("int bucket = k / 2 < 8 ? 8 : k / 2;", "int bucket = k / 2 < 9 ? 9 : k / 2;"),
    "mse_not_squared": ("row += d * d;", "row += fabs(d);"),
    "f32_sign_dropped": ("sg[i] = (uint8_t)(signbit(f) ? 1 : 0);", "sg[i] = 0;"),
    "f32_rounded_to_bf16_first": ("xv[i] = (double)f;",
                                  "{ uint32_t u_; memcpy(&u_, &f, 4); u_ = (u_ + 0x7fffu + ((u_ >> 16) & 1u)) & 0xffff0000u; "
                                  "float g_; memcpy(&g_, &u_, 4); xv[i] = (double)g_; }"),
    "mxfp8_exponent_bias": ("return (uint8_t)(((ex + 7) << 3) | mant);", "return (uint8_t)(((ex + 8) << 3) | mant);"),
    "mxfp8_mantissa_shift": ("int mant = ex <= 3 ? frac << (3 - ex) : frac >> (ex - 3);", "int mant = frac;"),
    "mxfp8_sign_lost": ("| ((code & 8) << 4));", "| ((code & 8) << 3));"),
    "mxfp8_scale_plus_3": ("(uint8_t)(meta[t * nblk + b] & 0xff);", "(uint8_t)((meta[t * nblk + b] & 0xff) + 3);"),
    "mxfp8_tile_rows_swapped": ("return tile * 512 + (r % 32) * 16 + (r / 32) * 4 + col % 4;",
                                "return tile * 512 + (r / 4) * 16 + (r % 4) * 4 + col % 4;"),
    "mxfp8_row_tiles_fastest": ("int64_t tile = (row / 128) * col_tiles + col / 4;",
                                "int64_t tile = (col / 4) * 3 + row / 128;"),
    "weights_absolute_error": ("err += diff * diff;", "err += fabs(diff);"),
    "weights_last_element_skipped": ("for (int i = 0; i < B; ++i) {\n          double diff", "for (int i = 0; i + 1 < B; ++i) {\n          double diff"),
    "weights_ties_to_highest": ("if (d == 0 || err < best_err) { best = d; best_err = err; }",
                                "if (d == 0 || err <= best_err) { best = d; best_err = err; }"),
    "weights_half_the_formatbook": ("for (int d = 0; d < 32; ++d) {\n        double err = 0.0;", "for (int d = 0; d < 16; ++d) {\n        double err = 0.0;"),
    "subformatbook_ties_to_highest": ("if (best < 0 || count[d] > count[best]) best = d;",
                                      "if (best < 0 || count[d] >= count[best]) best = d;"),
    "subformatbook_least_frequent": ("if (best < 0 || count[d] > count[best]) best = d;",
                                     "if (best < 0 || count[d] < count[best]) best = d;"),
    "subformatbook_buckets_ignored": ("if (!((stage1[k] >> d) & 1u)) continue;\n        if (best < 0 || count[d] > count[best])",
                                      "if (best < 0 || count[d] > count[best])"),
    "subformatbook_all_anchors_one_cluster": ("if (anchor_cluster[a] != c) continue;", ";"),
    "subformatbook_last_block_skipped": ("for (int64_t b = 0; b < nblk; ++b) count[", "for (int64_t b = 0; b + 1 < nblk; ++b) count["),
    "subformatbook_counts_scale_byte": ("count[(meta[t * nblk + b] >> 8) & 31] += 1;", "count[meta[t * nblk + b] & 31] += 1;"),
    "affine_two_roundings": ("y[t * C + c] = fmaf(xf, g, b);", "y[t * C + c] = (float)(xf * g) + b;"),
    "affine_one_plus_gain_exact": ("if (plus_one) g = 1.0f + g;\n      y[t * C + c] = fmaf(xf, g, b);",
                                   "y[t * C + c] = plus_one ? (float)((double)xf * (1.0 + (double)g) + (double)b) : fmaf(xf, g, b);"),
    "affine_plus_one_ignored": ("if (plus_one) g = 1.0f + g;\n      y[t * C + c] = fmaf(xf, g, b);",
                                "if (plus_one) g = g;\n      y[t * C + c] = fmaf(xf, g, b);"),
    "layernorm_plus_one_ignored": ("if (plus_one) g = 1.0f + g;\n      y[t * C + c] = fmaf(d[c] * rstd, g, bc);",
                                   "if (plus_one) g = g;\n      y[t * C + c] = fmaf(d[c] * rstd, g, bc);"),
    "affine_bias_of_next_channel": ("const float b = (float)bf16_to_double(bias[c]);",
                                    "const float b = (float)bf16_to_double(bias[c + 1 < C ? c + 1 : c]);"),
    "affine_ignores_row_stride": ("const float xf = (float)bf16_to_double(x[t * ld + c]);",
                                  "const float xf = (float)bf16_to_double(x[t * C + c]);"),
    "layernorm_block_sums_in_double": ("for (int i = 1; i < 32; ++i) s = s + (float)bf16_to_double(x[t * ld + b * 32 + i]);",
                                       "{ double s_ = s; for (int i = 1; i < 32; ++i) s_ += bf16_to_double(x[t * ld + b * 32 + i]); s = (float)s_; }"),
    "layernorm_butterfly_replaced_by_a_running_sum": ("  return v[0];\n}\n\nstatic float ln_row_total",
                                                     "  { float r_ = 0.0f; for (int i = 0; i < n; ++i) r_ += blocksum[i]; return r_; }\n}\n\nstatic float ln_row_total"),
    "layernorm_square_not_fused": ("q = fmaf(di, di, q);", "q = q + di * di;"),
    "layernorm_eps_dropped": ("const float rstd = 1.0f / sqrtf(var + eps);", "const float rstd = 1.0f / sqrtf(var);"),
    "layernorm_rsqrt_in_double": ("const float rstd = 1.0f / sqrtf(var + eps);", "const float rstd = (float)(1.0 / sqrt((double)var + (double)eps));"),
    "layernorm_variance_unbiased": ("const float var = ln_row_total(bs, nblk) / (float)C;", "const float var = ln_row_total(bs, nblk) / (float)(C - 1);"),
    "layernorm_modulation_two_roundings": ("y[t * C + c] = fmaf(d[c] * rstd, g, bc);", "y[t * C + c] = (d[c] * rstd) * g + bc;"),
    "layernorm_short_segment_padded_with_first_block": ("v[i] = i < n ? blocksum[i] : 0.0f;", "v[i] = i < n ? blocksum[i] : blocksum[0];"),
    "layernorm_segments_added_inexactly": ("total = total + ln_segment_butterfly(blocksum + b0, n);",
                                           "total = total * 1.0000001f + ln_segment_butterfly(blocksum + b0, n);"),
    "bf16_by_truncation": ("u += 0x7fffu + lsb;", "u += 0u * lsb;"),
    "bf16_ties_away_from_zero": ("u += 0x7fffu + lsb;", "u += 0x8000u + 0u * lsb;"),
    "bf16_ties_toward_zero": ("u += 0x7fffu + lsb;", "u += 0x7fffu + 0u * lsb;"),
    "salient_last_token_never_seen": ("int64_t t1 = t0 + tile < T ? t0 + tile : T, arg = t0;",
                                      "int64_t t1 = t0 + tile < T ? t0 + tile : T - 1, arg = t0;"),
    "residual_of_clamped_block_uses_unsaturated_value": (
        "float df = (float)(xv[i] - dequant_value(F, did, e, code[i]));",
        "float df = (float)(xv[i] - (fabs(xv[i]) >= ldexp(16.0, e - 3) ? xv[i] : dequant_value(F, did, e, code[i])));"),
    "f32_path_ignores_seda_mask": ("    const uint32_t allowed = row_mask(cluster_id, cluster_mask, n_clusters, t);\n    for (int64_t blk = 0; blk < nblk; ++blk) {\n      double xv[FB4O_MAXB];\n      uint8_t sg[FB4O_MAXB], code[FB4O_MAXB];\n      for (int i = 0; i < B; ++i) {\n        float f",
                                   "    const uint32_t allowed = 0xffffffffu;\n    for (int64_t blk = 0; blk < nblk; ++blk) {\n      double xv[FB4O_MAXB];\n      uint8_t sg[FB4O_MAXB], code[FB4O_MAXB];\n      for (int i = 0; i < B; ++i) {\n        float f"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch(name, tmp_path):
    old, new = MUTANTS[name]
    src = open(SRC).read()
    assert src.count(old) == 1, f"mutation site for {name} not unique/found"
    msrc = tmp_path / "mutant.c"
    msrc.write_text(src.replace(old, new))
    so = tmp_path / f"mutant_{name}.so"
    subprocess.check_call(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                           "-o", str(so), str(msrc), "-lm"])
    orc.use_library(str(so))
    caught = []
    try:
        for pin in pins.ALL_PINS:
            try:
                pin()
            except (AssertionError, ValueError, IndexError, StopIteration, ZeroDivisionError):
                caught.append(pin.__name__)
                break
    finally:
        orc.use_library(None)
    assert caught, f"no pin noticed the planted mistake '{name}'"
