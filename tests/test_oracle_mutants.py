"""The pins must be able to fail: plant one plausible mistake at a time in a copy of the
oracle (CPU only), rerun the pin tests against the copy and expect a failure."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "vl_oracle.c")

MUTANTS = [
    ("overlap uses <= (touching ranges collide)", "return a < b + wb && b < a + wa;", "return a <= b + wb && b < a + wa;"),
    ("range check off by one", "int unreal = s + w > p->P;", "int unreal = s + w >= p->P;"),
    ("definition compared with itself", "if (u == v) continue;", ""),
    ("kill dropped from the block transfer function",
     "uint8_t in = use[(size_t)b * V + v] | (o & !def[(size_t)b * V + v]);", "uint8_t in = use[(size_t)b * V + v] | o;"),
    ("reads after writes count as upward exposed", "if (!def[(size_t)b * V + v]) use[(size_t)b * V + v] = 1;",
     "use[(size_t)b * V + v] = 1;"),
    ("writes before reads in the backward walk",
     "for (uint32_t o = o0; o < o0 + nd; ++o) live[p->op_vreg[o]] = 0;\n            for (uint32_t o = o0 + nd; o < o1; ++o) live[p->op_vreg[o]] = 1;",
     "for (uint32_t o = o0 + nd; o < o1; ++o) live[p->op_vreg[o]] = 1;\n            for (uint32_t o = o0; o < o0 + nd; ++o) live[p->op_vreg[o]] = 0;"),
    ("duplicate source registers counted twice", "if (!dup) Q[nq++] = ta;", "Q[nq++] = ta;"),
    ("bank cost n instead of n-1", "bank += n - 1;", "bank += n;"),
    ("last occurrence wins", "if (T[v] < 0) T[v] = row[o];", "if (T[v] < 0 || 1) T[v] = row[o];"),
    ("co-defined vregs ignored", "if (in_live) continue;", "continue;"),
    ("Pass@k leaves out the k-th attempt", "if (attempts <= k[j]) summary[4 + j] += 1;",
     "if (attempts < k[j]) summary[4 + j] += 1;"),
    ("test cases that never pass counted among the attempts", "if (s[c].first_pass >= K[c]) continue; /* never passed */", ""),
    ("last passing attempt instead of the first", "if (s->first_pass == K) s->first_pass = k;", "s->first_pass = k;"),
    ("bank histogram charges the wrong bank", "if (bank_hist) bank_hist[Q[q] % p->B] += n - 1;",
     "if (bank_hist) bank_hist[Q[q] / p->B % p->B] += n - 1;"),
    ("own definitions kept in the occupied mask", "if (own) continue;", ""),
    ("occupied mask drops the last register of a tuple",
     "for (uint32_t r = (uint32_t)T[u]; r < (uint32_t)T[u] + p->vreg_width[u]; ++r)",
     "for (uint32_t r = (uint32_t)T[u]; r + 1 < (uint32_t)T[u] + p->vreg_width[u]; ++r)"),
    ("alignment tested on the end of the tuple", "if (p->vreg_align && s % p->vreg_align[v] != 0) unreal = 1;",
     "if (p->vreg_align && (s + w) % p->vreg_align[v] != 0) unreal = 1;"),
    ("class range closed at the top", "if (s < p->class_lo[c] || s + w > p->class_hi[c]) unreal = 1;",
     "if (s < p->class_lo[c] || s + w > p->class_hi[c] + 1) unreal = 1;"),
    ("class lower bound dropped", "if (s < p->class_lo[c] || s + w > p->class_hi[c]) unreal = 1;",
     "if (s + w > p->class_hi[c]) unreal = 1;"),
    ("dictionary entry reported at the first instruction of its block", "entry_instr[n] = i;",
     "entry_instr[n] = p->block_instr_off[b];"),
    ("every occurrence takes the entry of the last block that uses the vreg",
     "for (uint32_t e = dict_off[b]; e < dict_off[b + 1]; ++e) entry_of[dict_vreg[e]] = e;",
     "for (uint32_t e = 0; e < dict_off[p->n_blocks]; ++e) entry_of[dict_vreg[e]] = e;"),
    ("a vreg gets a dictionary entry only in the first block that uses it", "memset(seen, 0, (size_t)p->n_vregs + 1);\n        for",
     "if (b == 0) memset(seen, 0, (size_t)p->n_vregs + 1);\n        for"),
    ("reserved check leaves out the last register of a tuple", "for (uint32_t r = s; r < s + w && r < p->P; ++r)",
     "for (uint32_t r = s; r + 1 < s + w && r < p->P; ++r)"),
]


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_pins_catch_planted_mistake(tmp_path, name, old, new):
    text = open(SRC).read()
    assert text.count(old) >= 1, "mutation site vanished: " + name
    mutant = tmp_path / "vl_oracle_mutant.c"
    mutant.write_text(text.replace(old, new))        # every occurrence
    env = dict(os.environ, VL_ORACLE_MUTANT_SRC=str(mutant))
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_oracle_pins.py")],
                       cwd=ROOT, env=env, capture_output=True, text=True)
    assert r.returncode == 1, f"pins did not notice: {name}\n{r.stdout[-400:]}"
