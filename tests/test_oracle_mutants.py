"""Plant one plausible mistake at a time in a COPY of the CPU oracle and check
that the pins notice.  Nothing here touches a GPU or the CUDA library: the
mistakes are planted in the oracle's C source, compiled to a temporary shared
object, and the same pin functions are run against it."""
import os

import pytest

from oracle import gaf_oracle as orc
from pins import ALL_PINS

SRC = os.path.join(os.path.dirname(orc.__file__), "gaf_oracle.c")

# (name, text in the oracle, replacement)
MUTANTS = [
    ("strict_threshold", "int accept = (dc <= tau);", "int accept = (dc < tau);"),
    ("divide_by_k", "g[d] = g[d] / (double)c;", "g[d] = g[d] / (double)K;"),
    ("overwrite_not_add", "g[d] += elem(gi, d, dtype);", "g[d] = elem(gi, d, dtype);"),
    ("count_from_zero", "int32_t c = 1;", "int32_t c = 0;"),
    ("similarity_not_distance", "return 1.0 - cosv;", "return cosv;"),
    ("wrong_sign", "return 1.0 - cosv;", "return 1.0 + cosv;"),
    ("no_square_root", "cosv = p / (sqrt(na) * sqrt(nb));", "cosv = p / (na * nb);"),
    ("one_norm_only", "cosv = p / (sqrt(na) * sqrt(nb));", "cosv = p / sqrt(na);"),
    # (dropping the lower clamp is not listed: 1 - (-(1 + 2^-52)) rounds to 2 in
    #  binary64, so that change cannot be observed and is not a mistake)
    ("no_upper_clamp", "if (cosv > 1.0) cosv = 1.0;", ""),
    ("bf16_shift", "<< 16;", "<< 15;"),
    ("ignore_order", "int i = order ? order[t] : t;", "int i = t;"),
    ("ignore_seed", "int s = order ? order[0] : 0;", "int s = 0;"),
    ("mask_by_step", "mask[i] = 1;", "mask[t] = 1;"),
    ("dist_by_step", "dist[i] = dc;", "dist[t] = dc;"),
    ("test_against_seed", "p += v * g[d];", "p += v * elem(grads[s], d, dtype);"),
    ("norm_of_sum_dropped", "ng += g[d] * g[d];", "ng += v * v;"),
    ("norm_without_square", "ni += v * v;", "ni += v;"),
    ("cosdist_transposed_stats", "nx += a * a;", "nx += b * b;"),
    ("gram_not_mirrored", "gram[j * K + i] = p;", ""),
    ("gram_same_operand", "p += elem(grads[i], d, dtype) * elem(grads[j], d, dtype);",
     "p += elem(grads[i], d, dtype) * elem(grads[i], d, dtype);"),
    ("pairwise_wrong_norm", "gram[i * K + i], gram[j * K + j]);", "gram[i * K + i], gram[i * K + i]);"),
    ("forced_ignored", "if (forced && forced[t] >= 0) accept = forced[t];", ""),
    ("average_not_divided", "out[d] = sum / (double)K;", "out[d] = sum;"),
    ("bucket_offset_ignored", "sub[i] = (const char *)grads[i] + (size_t)lo * esize;", "sub[i] = (const char *)grads[i];"),
    ("bucket_mask_row", "mask + (size_t)b * K, dist + (size_t)b * K,", "mask, dist + (size_t)b * K,"),
    ("bucket_output_not_offset", "order, NULL, g + lo,", "order, NULL, g,"),
    ("ring_order_not_rotated", "for (int t = 0; t < K; ++t) order[t] = (s + t) % K;",
     "for (int t = 0; t < K; ++t) order[t] = t;"),
    ("ring_ties_to_last", "if (c > best_count) { best_count = c; best_seed = s; }",
     "if (c >= best_count) { best_count = c; best_seed = s; }"),
    ("ring_keeps_smallest", "if (c > best_count) { best_count = c; best_seed = s; }",
     "if (best_seed < 0 || c < best_count) { best_count = c; best_seed = s; }"),
]


@pytest.fixture
def restore_real_oracle():
    yield
    orc.use_library(None)


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_pins_catch_planted_mistake(name, old, new, tmp_path, restore_real_oracle):
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation site for {name} must be unique"
    c_file = tmp_path / f"mutant_{name}.c"
    c_file.write_text(text.replace(old, new))
    lib = orc.compile_c(str(c_file), str(tmp_path / f"mutant_{name}.so"))
    orc.use_library(lib)
    caught = None
    for pin in ALL_PINS:
        try:
            pin()
        except AssertionError:
            caught = pin.__name__
            break
    assert caught is not None, f"no pin notices the mistake '{name}'"
