"""Plant one mistake at a time in a copy of the oracle's source (CPU only) and require that
at least one pin notices.  This measures the pins, not the oracle: a mutant that survives
means a plausible mistake in the oracle would go unseen."""
import os
import subprocess

import pytest

import oracle_pins as pins
from oracle import apms_oracle as ao
from oracle import build as ob

MUTANTS = [
    ("sign_of_zero", "if (z[j] >= 0.0f) bits", "if (z[j] > 0.0f) bits"),
    ("msb_first_bits", "(uint32_t)1 << (j % 32);", "(uint32_t)1 << (31 - j % 32);"),
    ("scale_not_normalised", "(float)sqrt(acc / (double)L)", "(float)sqrt(acc)"),
    ("scale_l1_instead_of_l2", "else                                    acc += (double)z[j] * (double)z[j];",
     "else                                    acc += fabs((double)z[j]);"),
    ("worker_error_sign", "e[j] = z[j] - qi[j];", "e[j] = z[j] + qi[j];"),
    ("worker_error_dropped", "z[j] = mi + e[j];", "z[j] = mi;"),
    ("no_average", "z[j] = acc / (float)n + o->ebar[lo + j];", "z[j] = acc + o->ebar[lo + j];"),
    ("server_error_dropped", "z[j] = acc / (float)n + o->ebar[lo + j];", "z[j] = acc / (float)n;"),
    ("server_error_not_updated", "o->ebar[lo + j] = z[j] - qb[j];", "o->ebar[lo + j] = z[j];"),
    ("momentum_not_replaced", "o->m[lo + j] = qb[j];", "o->m[lo + j] = z[j];"),
    ("precondition_without_sqrt", "(sqrtf(o->v[lo + j]) + o->eps)", "(o->v[lo + j] + o->eps)"),
    ("update_sign", "o->x[lo + j] - (o->lr * o->m[lo + j])", "o->x[lo + j] + (o->lr * o->m[lo + j])"),
    ("beta_swapped", "fmaf(o->beta1, o->m[lo + j], omb1 * g[i][lo + j])",
     "fmaf(omb1, o->m[lo + j], o->beta1 * g[i][lo + j])"),
    ("all_workers_use_gradient_0", "omb1 * g[i][lo + j]", "omb1 * g[0][lo + j]"),
    ("scale_slot", "o->s + (size_t)i * (size_t)o->C + c;", "o->s + (size_t)i * (size_t)o->C;"),
    ("adam_no_sqrt", "(sqrtf(vhat) + o->eps)", "(vhat + o->eps)"),
    ("adam_no_bias_correction_m", "const float mhat = o->m[j] / bc1;", "const float mhat = o->m[j];"),
    ("adam_no_bias_correction_v", "const float vhat = o->v[j] / bc2;", "const float vhat = o->v[j];"),
    ("adam_gradient_not_averaged", "const float gbar = gs / (float)o->n;", "const float gbar = gs;"),
    ("adam_v_not_squared", "omb2 * (gbar * gbar)", "omb2 * gbar"),
    ("adam_bc2_uses_beta1", "pow((double)o->beta2, (double)o->t)", "pow((double)o->beta1, (double)o->t)"),
    ("v_keeps_updating", "o->x[lo + j] = o->x[lo + j] - (o->lr * o->m[lo + j])",
     "o->v[lo + j] = 0.999f * o->v[lo + j]; o->x[lo + j] = o->x[lo + j] - (o->lr * o->m[lo + j])"),
    ("gradient_variant_sends_momentum", "? g[i][lo + j]                                      /* the gradient itself is sent */",
     "? fmaf(o->beta1, o->m[lo + j], omb1 * g[i][lo + j])"),
    ("gradient_variant_momentum_replaced", "o->m[lo + j] = fmaf(o->beta1, o->m[lo + j], omb1 * qb[j]);", "o->m[lo + j] = qb[j];"),
    ("gradient_variant_betas_swapped", "fmaf(o->beta1, o->m[lo + j], omb1 * qb[j])", "fmaf(omb1, o->m[lo + j], o->beta1 * qb[j])"),
    ("gradient_variant_update_uses_gradient", "else                                       o->m[lo + j] = qb[j];",
     "else                                       o->m[lo + j] = qb[j];\n        if (o->variant == ORACLE_VARIANT_GRADIENT) { o->x[lo + j] = o->x[lo + j] - (o->lr * qb[j]) / (sqrtf(o->v[lo + j]) + o->eps); continue; }"),
    ("topk_keeps_smallest", "if (x->key != y->key) return x->key > y->key ? -1 : 1;", "if (x->key != y->key) return x->key < y->key ? -1 : 1;"),
    ("topk_ties_to_higher_index", "return x->idx < y->idx ? -1 : (x->idx > y->idx ? 1 : 0);", "return x->idx > y->idx ? -1 : (x->idx < y->idx ? 1 : 0);"),
    ("topk_signed_comparison", "items[j].key = bits & 0x7fffffffu;", "items[j].key = bits;"),
    ("topk_one_too_many", "for (int64_t r = 0; r < K && r < L; ++r)", "for (int64_t r = 0; r <= K && r < L; ++r)"),
    ("topk_count_floor", "int64_t K = (int64_t)ceil(frac * (double)L);", "int64_t K = (int64_t)floor(frac * (double)L);"),
    ("topk_server_not_compressed", "apms_oracle_compress_topk(z, L, apms_oracle_topk_count(o->topk_frac, L), qb, o->selbar + lo);",
     "memcpy(qb, z, (size_t)L * sizeof(float));"),
    ("server_uses_last_worker_only", "acc += q[(size_t)i * (size_t)L + j];",
     "acc = q[(size_t)i * (size_t)L + j] * (float)n;"),
]


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(tmp_path, name, old, new):
    src = open(ob.SRC).read()
    assert src.count(old) == 1, f"mutation site for {name} not unique: {src.count(old)}"
    msrc = tmp_path / "mutant.c"
    msrc.write_text(src.replace(old, new))
    mlib = str(tmp_path / "libmutant.so")
    ob.build(force=True, src=str(msrc), lib=mlib)
    library = ao.lib(mlib)
    caught = []
    for check in pins.ALL_CHECKS:
        try:
            check(library)
        except AssertionError:
            caught.append(check.__name__)
            break
    assert caught, f"no pin noticed the planted mistake '{name}'"
