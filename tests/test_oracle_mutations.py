"""Plant plausible mistakes in a COPY of the oracle (on the CPU) and check that
the pin suite notices every one of them: a pin that nothing can fail pins nothing."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "tuna_oracle.c")

# (name, text in the oracle, replacement)
MUTATIONS = [
    ("mirror_direction",
     "int to = (int)((p + dist) % P);", "int to = (int)(((p - dist) % P + P) % P);"),
    ("mirror_direction_recv",
     "int from = (int)(((q - dist) % P + P) % P);", "int from = (int)((q + dist) % P);"),
    ("printed_final_condition",          # Algorithm 1's listing: "if (i % r^x == 0) receive into R"
     "int final = o < rx * r;", "int final = (o % rx) == 0;"),
    ("keep_rounds_beyond_P",
     "      if ((int64_t)z * ipow(r, x) >= P) continue;", "      if (0) continue;"),
    ("ceiling_in_tmap",
     "while (ipow(r, dx + 1) <= o) dx++;", "while (ipow(r, dx) < o) dx++;"),
    ("tmap_forgets_self_block",
     "return o - 1 - dx * (r - 1) - dz;", "return o - dx * (r - 1) - dz;"),
    ("transposed_rdispls",
     "rdispls[(int64_t)q * P + src_rank]) * elem, m->data + at,",
     "rdispls[(int64_t)src_rank * P + q]) * elem, m->data + at,"),
    ("transposed_counts_in_definition",
     "int64_t n = counts[(int64_t)s * P + d] * elem;", "int64_t n = counts[(int64_t)d * P + s] * elem;"),
    ("digit_test_always_one",            # "whose x-th digit is 1"
     "if (digit_of(o, r, x) == z) out[n++] = o;", "if (digit_of(o, r, x) == 1) out[n++] = o;"),
    ("hier_wrong_group_partner",
     "int from = (int)(((n - dist) % N + N) % N) * Q + q;", "int from = (int)((n + dist) % N) * Q + q;"),
    ("hier_own_group_blocks_kept_in_T",
     "if (local_final && i == n) {", "if (0) {"),
    ("compaction_lists_parts_by_local_offset",   # Sec. IV-B: parts in ascending source local id
     "        int64_t nb = sz[(int64_t)p * P + i * Q + jo];\n        usz[((int64_t)p * N + io) * Q + qs] = nb;",
     "        int64_t nb = sz[(int64_t)p * P + i * Q + jo];\n        usz[((int64_t)p * N + io) * Q + jo] = nb;"),
    ("staggered_sends_the_wrong_way",
     "          int ndst = ((n - gi) % N + N) % N;\n          if (ndst == n) continue;\n          active = 1;",
     "          int ndst = (n + gi) % N;\n          if (ndst == n) continue;\n          active = 1;"),
    ("staggered_mirrored_both_ways",     # consistent, but not the direction Algorithm 2 prints
     ("int ndst = ((n - gi) % N + N) % N;", "int nsrc = (n + gi) % N;"),
     ("int ndst = (n + gi) % N;", "int nsrc = ((n - gi) % N + N) % N;")),
    ("staggered_owner_index_is_receiver",
     "          int jo = ((q - gr) % Q + Q) % Q;\n          int64_t nb = sz[(int64_t)p * P + ndst * Q + jo];",
     "          int jo = gr;\n          int64_t nb = sz[(int64_t)p * P + ndst * Q + jo];"),
    ("rows_maps_swapped",
     "int64_t from = gather ? gather[js] : js;\n        int64_t to = scatter ? scatter[jr] : jr;",
     "int64_t from = gather ? gather[jr] : js;\n        int64_t to = scatter ? scatter[js] : jr;"),
    ("scan_inclusive",
     "      out[s * seglen + i] = run;\n      run += v;", "      run += v;\n      out[s * seglen + i] = run;"),
    ("dropped_self_block",
     "  /* the self block never travels */\n  for (int p = 0; p < P; p++)\n    memcpy(",
     "  /* the self block never travels */\n  for (int p = 0; p < 0; p++)\n    memcpy("),
]


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_pins_catch_a_planted_mistake(tmp_path, name, old, new):
    text = open(SRC).read()
    olds, news = (old, new) if isinstance(old, tuple) else ((old,), (new,))
    for o, n in zip(olds, news):
        assert text.count(o) >= 1, f"mutation {name} no longer applies: update it"
        text = text.replace(o, n, 1)
    mutated = tmp_path / "tuna_oracle_mutated.c"
    mutated.write_text(text)
    env = dict(os.environ, TUNA_ORACLE_SOURCE=str(mutated))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                        "-x", "-q", "-p", "no:cacheprovider"], cwd=ROOT, env=env, capture_output=True,
                       text=True, timeout=600)
    assert r.returncode != 0, f"the pins did not notice mutation {name}"
