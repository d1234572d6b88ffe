"""Strength of the oracle's pins: every plausible mistake planted in a copy of the
oracle source (a dropped term, a wrong factor, index or comparison, a swapped
operand) must make at least one pin of tests/test_oracle_pins.py fail.  The mistakes
are planted on the CPU, in a temporary copy; the committed oracle is untouched."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "llmem_oracle.c")

# (name, text to find, replacement); each `find` must occur exactly `count` times
MUTANTS = [
    ("os_drops_variance", "shard((B32 + B32) * z->hh_p, c)", "shard(B32 * z->hh_p, c)", 1),
    ("os_embedding_half", "shard((B32 + B32) * z->tok_p, c)", "shard(B32 * z->tok_p, c)", 1),
    ("p32_as_fp16", "z->p32_chunk = shard(B32 * cs, c);", "z->p32_chunk = shard(B16 * cs, c);", 1),
    ("p16_embed_double", "z->p16_embed = shard(B16 * z->embed_p, c);", "z->p16_embed = shard(B32 * z->embed_p, c);", 1),
    ("shift_full_length", "z->shift = bs * (sl - 1) * V", "z->shift = bs * sl * V", 1),
    ("single_shift_copy", "    emit(s, +1, z->shift);\n    emit(s, +1, z->shift);", "    emit(s, +1, z->shift);", 1),
    ("back_factor", "ceil_div(z->out * (t - 1), t)", "ceil_div(z->out * t, t)", 1),
    ("back_degree_always_gpu_n", "u128 t = (c->method == M_TP) ? c->gpu_n : c->tp_n;", "u128 t = c->gpu_n;", 1),
    ("dptp_gather_keeps_all", "return whole - (whole * c->tp_n) / c->gpu_n - kept;", "return whole - kept;", 1),
    ("adp_gather_double", "if (c->method == M_ADP) return whole - kept;", "if (c->method == M_ADP) return whole;", 1),
    ("os_in_last_iteration", "if (it == 1) {", "if (it == c->iters) {", 1),
    ("round_down", "static u128 page_round(u128 x) { return ceil_div(x, CU_P) * CU_P; }",
     "static u128 page_round(u128 x) { return x / CU_P * CU_P; }", 1),
    ("page_one_mib", "#define CU_P ((u128)2 * 1024 * 1024)", "#define CU_P ((u128)1 * 1024 * 1024)", 1),
    ("chunks_floor", "z->C = ceil_div(z->other_p, (u128)c->chunk_elems);", "z->C = z->other_p / (u128)c->chunk_elems;", 1),
    ("embed_without_positions", "z->embed_p = z->tok_p + z->pos_p;", "z->embed_p = z->tok_p;", 1),
    ("one_norm_per_layer", "u128 norm_p = 2 * H * (1 + bias);", "u128 norm_p = H * (1 + bias);", 1),
    ("ffn_bias_count", "bias * (4 * H + (nffn - 1) * F + H)", "bias * (4 * H + nffn * F + H)", 1),
    ("lm_head_dropped", "u128 off = (u128)c->base_bytes + z.lm_p;\n  if (off >= BYTES_LIMIT) return ST_OVERFLOW;\n  *offset_out",
     "u128 off = (u128)c->base_bytes;\n  if (off >= BYTES_LIMIT) return ST_OVERFLOW;\n  *offset_out", 1),
    ("tie_prefers_later", "if (eval2[i] > eval2[idx]) idx = i;", "if (eval2[i] >= eval2[idx]) idx = i;", 1),
    ("cdp_score_factor", "eval2[0] = (int64_t)bs_list[0] * n * 3;", "eval2[0] = (int64_t)bs_list[0] * n * 2;", 1),
    ("offload_predicate_slot", "(flags & SELECT_ALLZERO) ? any : (eval2[2] != 0)", "(flags & SELECT_ALLZERO) ? any : (eval2[1] != 0)", 1),
    ("dp_degree", "(n / tp_n) * 2 : 0;", "(int64_t)tp_n * 2 : 0;", 1),
    ("fits_is_strict", "if (e != ST_OK || peak > capacity) break; /* m_peak > m_total */",
     "if (e != ST_OK || peak >= capacity) break;", 1),
    ("bisect_fits_is_strict", "if (e == ST_OK && peak <= capacity)", "if (e == ST_OK && peak < capacity)", 1),
    ("last_arg_max", "if (arg < 0 || run > best) {", "if (arg < 0 || run >= best) {", 1),
    ("gated_tensor_count", "z->K = c->ffn_kind ? 7 : 6;", "z->K = c->ffn_kind ? 8 : 6;", 1),
    ("attention_tensor_count", "emit(s, +1, k < 4 ? z->os_hh : z->os_hf);", "emit(s, +1, k < 3 ? z->os_hh : z->os_hf);", 1),
    ("cdp_sharded", "return c->method == M_CDP ? bytes : ceil_div(bytes, c->gpu_n);", "return ceil_div(bytes, c->gpu_n);", 1),
    ("outputs_fp32", "z->out = bs * sl * H * B16;", "z->out = bs * sl * H * B32;", 1),
    ("embedding_outputs_missing", "for (int64_t i = 0; i < z->e_n; ++i) emit(s, +1, z->out);",
     "for (int64_t i = 0; i + 1 < z->e_n; ++i) emit(s, +1, z->out);", 1),
    ("scores_without_heads", "z->act_attn = bs * (u128)c->heads * sl * sl * B16;", "z->act_attn = bs * sl * sl * B16;", 1),
    ("one_attention_matrix", "static const int plain[14] = {0, 0, 0, 0, 1, 1, 0,", "static const int plain[14] = {0, 0, 0, 0, 1, 0, 0,", 1),
    ("gated_like_plain", "static const int gated[16] = {0, 0, 0, 0, 1, 1, 0, 0, 0, 0, 2, 2, 2, 2, 0, 0};",
     "static const int gated[16] = {0, 0, 0, 0, 1, 1, 0, 0, 0, 0, 2, 2, 0, 0, 0, 0};", 1),
    ("operator_frees_in_forward_order", "for (int k = z->n_ops - 1; k >= 0; --k) emit(s, -1, op_size(z, k));",
     "for (int k = 0; k < z->n_ops; ++k) emit(s, -1, op_size(z, k));", 1),
    ("ffn_outputs_hidden_sized", "z->act_ffn = bs * sl * F * B16;", "z->act_ffn = bs * sl * H * B16;", 1),
    ("collapsed_single_iteration", "u128 rel = c->iters >= 2 ? later : (first > after ? first : after);",
     "u128 rel = later;", 1),
    ("collapsed_os_count", "(u128)z->L * (4 * page_round(z->os_hh) + (u128)(z->K - 4) * page_round(z->os_hf));",
     "(u128)z->L * (4 * page_round(z->os_hh) + (u128)(z->K - 5) * page_round(z->os_hf));", 1),
    ("tp_without_backward_buffers", "z->tpback = (c->method == M_TP || c->method == M_DPTP);", "z->tpback = (c->method == M_DPTP);", 1),
    ("segmented_tie_prefers_later", "if (score2 > best_score) { /* strict: the first of equals stays */",
     "if (score2 >= best_score && score2 > 0) {", 1),
    ("segmented_dp_degree", "score2 = (i128)2 * b * (c->gpu_n / c->tp_n);", "score2 = (i128)2 * b * c->tp_n;", 1),
    ("segmented_cdp_factor", "score2 = (i128)3 * b * c->gpu_n;", "score2 = (i128)2 * b * c->gpu_n;", 1),
    ("chunk_search_last_minimum", "if (best_cs < 0 || waste < best_waste) { /* strict: the first of equals stays */",
     "if (best_cs < 0 || waste <= best_waste) {", 1),
    ("chunk_search_floor", "u128 waste = ceil_div(z.other_p, cs) * cs - z.other_p;",
     "u128 waste = (z.other_p / cs + 1) * cs - z.other_p;", 1),
    ("dnn_align_down", "static u128 align512(u128 x) { return ceil_div(x, DNN_ALIGN) * DNN_ALIGN; }",
     "static u128 align512(u128 x) { return x / DNN_ALIGN * DNN_ALIGN; }", 1),
    ("dnn_buffer_dropped", "  emit(s, +1, DNN_BUFFER);\n", "", 1),
    ("dnn_weights_fp32", "emit(s, +1, B16 * (k < 4 ? z->hh_p : z->hf_p));", "emit(s, +1, B32 * (k < 4 ? z->hh_p : z->hf_p));", 1),
    ("dnn_bias_count", "int small = 2 + (int)bias * 7, wide = (int)bias * (z->K - 5);", "int small = 2 + (int)bias * 6, wide = (int)bias * (z->K - 5);", 1),
    ("dnn_operator_kind", "for (int k = 0; k < z->n_ops; ++k) emit(s, +1, op_size(z, k));\n  emit(s, +1, z->logit);",
     "for (int k = 0; k < z->n_ops; ++k) emit(s, +1, op_size(z, z->op_kind[k]));\n  emit(s, +1, z->logit);", 1),
    ("dnn_accepts_sharded_methods", "  if (c->method != M_CDP) return ST_COMBO;\n  return ST_OK;", "  return ST_OK;", 1),
    ("frees_forgotten_gather", "      for (int64_t j = 0; j < C; ++j) emit(s, -1, z->gat_chunk);\n", "", 1),
]


def _run_pins(lib_path):
    env = dict(os.environ, LLMEM_ORACLE_LIB=lib_path)
    return subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                           "-x", "-q", "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True, text=True)


def _compile(text, out_dir, name):
    c_path = os.path.join(out_dir, name + ".c")
    so_path = os.path.join(out_dir, name + ".so")
    open(c_path, "w").write(text)
    subprocess.check_call(["gcc", "-O1", "-std=c11", "-shared", "-fPIC", "-o", so_path, c_path, "-lpthread"])
    return so_path


def test_unmodified_copy_passes(tmp_path):
    so = _compile(open(SRC).read(), str(tmp_path), "pristine")
    r = _run_pins(so)
    assert r.returncode == 0, r.stdout[-2000:]


@pytest.mark.parametrize("name,find,repl,count", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(tmp_path, name, find, repl, count):
    src = open(SRC).read()
    assert src.count(find) == count, f"mutation site of {name} not found exactly {count} time(s)"
    so = _compile(src.replace(find, repl), str(tmp_path), name)
    r = _run_pins(so)
    assert r.returncode != 0, f"no pin notices the planted mistake '{name}'"
    assert " failed" in r.stdout or "Error" in r.stdout or "error" in r.stdout
