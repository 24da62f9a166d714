"""Do the pins notice a mistake?  Each case plants ONE plausible error in a copy of
the oracle's C source (on the CPU, never in the product), builds it, and requires
that at least one pin of tests/oracle_pins.py fails on it.  The committed source
must contain every text that is replaced, so the list cannot silently go stale."""
import os
import shutil

import pytest

import oracle
import oracle.build
import oracle_pins

ORACLE_DIR = os.path.dirname(os.path.abspath(oracle.build.__file__))

# (name, file, committed text, mutated text)
MUTANTS = [
    ("block_one_too_long", "def_oracle.c", "return offset < k;", "return offset <= k;"),
    ("block_does_not_wrap", "def_oracle.c", "if (offset < 0) offset += d;", ""),
    ("block_before_start", "def_oracle.c", "int64_t offset = j - s;", "int64_t offset = s - j;"),
    ("error_sign", "def_oracle_body.inc", "e_w[i] = p[i] - Cp_w[i];", "e_w[i] = p[i] + Cp_w[i];"),
    ("error_keeps_everything", "def_oracle_body.inc", "e_w[i] = p[i] - Cp_w[i];", "e_w[i] = p[i];"),
    ("update_sign", "def_oracle_body.inc", "x[i] = x[i] - C_pt;", "x[i] = x[i] + C_pt;"),
    ("no_average", "def_oracle_body.inc", "REAL C_pt = sum / (REAL)W;", "REAL C_pt = sum;"),
    ("worker_dropped", "def_oracle_body.inc",
     "for (int64_t w = 1; w < W; ++w)                     /* workers added",
     "for (int64_t w = 2; w < W; ++w)                     /* workers added"),
    ("momentum_operands_swapped", "def_oracle_body.inc",
     "m_w[i] = FMA(mu, m_w[i], g_w[i]);", "m_w[i] = FMA(mu, g_w[i], m_w[i]);"),
    ("momentum_not_used_in_p", "def_oracle_body.inc",
     "p[i] = FMA(eta, m_w[i], e_w[i]);", "p[i] = FMA(eta, g_w[i], e_w[i]);"),
    ("momentum_eta_misplaced", "def_oracle_body.inc",
     "m_w[i] = FMA(mu, m_w[i], g_w[i]);", "m_w[i] = FMA(mu, m_w[i], eta * g_w[i]);"),
    ("error_term_dropped", "def_oracle_body.inc",
     "p[i] = FMA(eta, g_w[i], e_w[i]);            /* p_{k,t} = eta g", "p[i] = eta * g_w[i];            /* p_{k,t} = eta g"),
    ("eta_dropped", "def_oracle_body.inc",
     "p[i] = FMA(eta, g_w[i], e_w[i]);            /* p_{k,t} = eta g", "p[i] = g_w[i] + e_w[i];            /* p_{k,t} = eta g"),
    ("scale_compressor_identity", "def_oracle_body.inc", "out[i] = delta * in[i];", "out[i] = in[i];"),
    ("detach_sign", "def_oracle_body.inc", "FMA(-lambda, e_w[i], x[i])", "FMA(lambda, e_w[i], x[i])"),
    ("detach_ignores_lambda", "def_oracle_body.inc", "FMA(-lambda, e_w[i], x[i])", "x[i] - e_w[i]"),
    ("output_sign", "def_oracle_body.inc", "out[i] = x[i] - sum / (REAL)W;", "out[i] = x[i] + sum / (REAL)W;"),
    ("output_not_averaged", "def_oracle_body.inc", "out[i] = x[i] - sum / (REAL)W;", "out[i] = x[i] - sum;"),
    ("defa_returns_y", "def_oracle_body.inc", "if (variant == DEF_ORACLE_VARIANT_DEF) {",
     "if (variant != DEF_ORACLE_VARIANT_EF) {"),
    ("stats_mean_not_divided", "def_oracle_body.inc", "e_t /= (double)W;", ""),
    ("stats_detach_sign", "def_oracle_body.inc", "double diff = e_t - (double)lambda * e_k;", "double diff = e_t + (double)lambda * e_k;"),
    ("stats_lambda_ignored", "def_oracle_body.inc", "double diff = e_t - (double)lambda * e_k;", "double diff = e_t - e_k;"),
    ("stats_not_averaged", "def_oracle_body.inc", "out[0] = mean_sq / (double)W;", "out[0] = mean_sq;"),
    ("stats_detached_not_averaged", "def_oracle_body.inc", "out[2] = detached / (double)W;", "out[2] = detached;"),
    ("philox_multipliers_swapped", "def_oracle.c",
     "MUL0 = 0xD2511F53u, MUL1 = 0xCD9E8D57u", "MUL0 = 0xCD9E8D57u, MUL1 = 0xD2511F53u"),
    ("philox_wrong_high_half", "def_oracle.c", "uint32_t n0 = hi1 ^ c1 ^ k0;", "uint32_t n0 = hi0 ^ c1 ^ k0;"),
    ("philox_key_bumped_early", "def_oracle.c", "if (r > 0) { k0 += WEYL0; k1 += WEYL1; }",
     "{ k0 += WEYL0; k1 += WEYL1; }"),
    ("philox_weyl_swapped", "def_oracle.c", "WEYL0 = 0x9E3779B9u, WEYL1 = 0xBB67AE85u",
     "WEYL0 = 0xBB67AE85u, WEYL1 = 0x9E3779B9u"),
    ("start_by_modulo", "def_oracle.c", "return (int64_t)(uint64_t)(wide >> 64);", "return (int64_t)(r % (uint64_t)d);"),
    ("start_uses_wrong_words", "def_oracle.c", "(uint64_t)out[0] | ((uint64_t)out[1] << 32)",
     "(uint64_t)out[2] | ((uint64_t)out[3] << 32)"),
    ("start_nine_rounds", "def_oracle.c", "def_oracle_philox4x32(ctr, key, 10, out);",
     "def_oracle_philox4x32(ctr, key, 9, out);"),
]


def _failing_pins(o):
    failed = []
    for name, pin in oracle_pins.ALL_PINS:
        try:
            pin(o)
        except AssertionError:
            failed.append(name)
    return failed


@pytest.mark.parametrize("name,fname,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_mutant_is_caught(tmp_path, name, fname, old, new):
    for f in oracle.build.DEPENDS:
        shutil.copy(os.path.join(ORACLE_DIR, f), tmp_path / f)
    text = (tmp_path / fname).read_text()
    assert text.count(old) == 1, "the committed oracle no longer contains exactly one %r" % old
    (tmp_path / fname).write_text(text.replace(old, new))
    lib = oracle.build.build(force=True, lib=str(tmp_path / "libdef_oracle_mutant.so"),
                             source_dir=str(tmp_path), extra_flags=["-w"])
    failed = _failing_pins(oracle.Oracle(lib))
    assert failed, "no pin notices the planted mistake %r" % name


def test_committed_oracle_passes_every_pin():
    assert _failing_pins(oracle.default()) == []
