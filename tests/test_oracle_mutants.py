"""Do the pins bite?  Each case plants ONE plausible mistake in a copy of the oracle's C source (a dropped
update, an off-by-one, a wrong comparison, a transposed index), compiles the copy, and runs the oracle's pin
tests against it in a child process.  Every planted mistake must make at least one pin fail; the unchanged
source must pass the same run (so a failure is the pins' verdict and not the harness').  CPU only; nothing
here touches the CUDA path.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent
SOURCE = ROOT / "oracle" / "sam_oracle.c"
BATTERY = ["tests/test_oracle_pins.py", "tests/test_oracle_dynamic.py", "tests/test_oracle_options.py"]

# (name, text in the source, what the mistake puts there).  Not in the list, because it changes nothing: a miss at
# the root that leaves the matched length alone - whenever the walk stands at the root that length is already 0.
MUTANTS = [
    ("clone takes the current position instead of the original's first occurrence",
     "a->st[clone].firstpos = sq->firstpos;", "a->st[clone].firstpos = i;"),
    ("clone keeps the original's length",
     "a->st[clone].len = a->st[p].len + 1;", "a->st[clone].len = sq->len;"),
    ("clone's suffix link goes to the root",
     "a->st[clone].link = sq->link;", "a->st[clone].link = 0;"),
    ("only the first transition is redirected to the clone",
     "while (p != -1 && edge_get(&a->st[p], c) == q) {", "if (p != -1 && edge_get(&a->st[p], c) == q) {"),
    ("the split state's suffix link is not moved to the clone",
     "            a->st[q].link = clone;\n", ""),
    ("new state linked to the root although a continuation state exists",
     "a->st[cur].link = q;", "a->st[cur].link = 0;"),
    ("new state's length not advanced",
     "a->st[cur].len = a->st[a->last].len + 1;", "a->st[cur].len = a->st[a->last].len;"),
    ("a miss shortens the match by one instead of to the link's length",
     "            L = a->st[s].len;\n", "            L = L - 1;\n"),
    ("after a miss the token is dropped instead of being retried from the suffix link",
     "            L = a->st[s].len;\n", "            L = a->st[s].len; break;\n"),
    ("a miss at the root is reported as a match of one token",
     "if (s == 0) { L = 0; break; }", "if (s == 0) { L = 1; break; }"),
    ("draft starts at the last matched token",
     "int64_t p = (int64_t)a->st[state].firstpos + 1;", "int64_t p = (int64_t)a->st[state].firstpos;"),
    ("draft runs across a separator",
     "        if (is_separator(corpus[p + j], seps, n_sep)) break;\n", ""),
    ("draft needs one token more than min_match",
     "if (matched_len < min_match) return 0;", "if (matched_len <= min_match) return 0;"),
    ("draft may run one token past the end of the text",
     "if (p + j >= n) break;", "if (p + j > n) break;"),
    ("argmax keeps the last of equal maxima",
     "if (x > best) { best = x; idx = v; }", "if (x >= best) { best = x; idx = v; }"),
    ("argmax compares bit patterns instead of values",
     "    uint32_t u = (uint32_t)b << 16;\n    float f;\n    memcpy(&f, &u, sizeof f);\n    return f;",
     "    return (float)b;"),
    ("accept compares draft j with row j+1",
     "while (a < n_draft && drafts[a] == argmax_row[a]) {", "while (a < n_draft && drafts[a] == argmax_row[a + 1]) {"),
    ("accept forgets the model's own token",
     "    accepted[a] = argmax_row[a];\n    return a + 1;", "    return a;"),
    ("renormalize stops one link early",
     "while (s != 0 && matched_len <= a->st[a->st[s].link].len) s = a->st[s].link;",
     "while (s != 0 && matched_len < a->st[a->st[s].link].len) s = a->st[s].link;"),
    ("accepted-draft counter includes the model's own token",
     "counters[3] += n_accepted[b] - 1;", "counters[3] += n_accepted[b];"),
    ("row skipping also skips the row that gives the model's own token",
     "if ((flags & ORACLE_SKIP_UNUSED_ROWS) && j > nd) { am[j] = -1; continue; }",
     "if ((flags & ORACLE_SKIP_UNUSED_ROWS) && j >= nd) { am[j] = -1; continue; }"),
    ("speculation switched off still emits a draft",
     "        if (flags & ORACLE_NO_SPECULATION) {\n            for (int32_t j = 0; j < K; j++) nx[j] = -1;\n"
     "            next_n_draft[b] = 0;\n        } else {",
     "        if (0) {\n            for (int32_t j = 0; j < K; j++) nx[j] = -1;\n"
     "            next_n_draft[b] = 0;\n        } else {"),
    ("the counter-driven switch speculates on a tie between tokens and cost",
     "return (double)accepted * (double)K > (cost_ratio - 1.0) * (double)(rows - passes);",
     "return (double)accepted * (double)K >= (cost_ratio - 1.0) * (double)(rows - passes);"),
    ("the counter-driven switch charges the first row of a pass as an extra row",
     "return (double)accepted * (double)K > (cost_ratio - 1.0) * (double)(rows - passes);",
     "return (double)accepted * (double)K > (cost_ratio - 1.0) * (double)(rows);"),
    ("the counter-driven switch forgets that the extra cost is spread over K rows",
     "return (double)accepted * (double)K > (cost_ratio - 1.0) * (double)(rows - passes);",
     "return (double)accepted > (cost_ratio - 1.0) * (double)(rows - passes);"),
    ("the counter-driven switch compares all committed tokens with the extra cost",
     "const int64_t passes = counters[0], accepted = counters[3], rows = counters[5];",
     "const int64_t passes = counters[0], accepted = counters[1], rows = counters[5];"),
]

_CHILD = r"""
import pathlib, sys
sys.path.insert(0, {root!r})
import oracle
oracle._SRC = pathlib.Path({src!r})
oracle._SO = pathlib.Path({so!r})
oracle._lib = None
import pytest
sys.exit(pytest.main(["-x", "-q", "-p", "no:cacheprovider"] + {battery!r}))
"""


def _compile(src: Path, so: Path) -> None:
    subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", str(so), str(src)])


def _run_battery(src: Path, so: Path) -> int:
    """Exit code of the pin tests run against the library at `so`: 0 = all passed, 1 = some pin failed."""
    code = _CHILD.format(root=str(ROOT), src=str(src), so=str(so), battery=BATTERY)
    env = dict(os.environ, OMP_NUM_THREADS="1")
    try:
        p = subprocess.run([sys.executable, "-c", code], cwd=str(ROOT), env=env, stdout=subprocess.PIPE,
                           stderr=subprocess.STDOUT, timeout=600)
    except subprocess.TimeoutExpired:
        return 1                                            # a pin that never returns has not passed
    if p.returncode not in (0, 1):
        raise RuntimeError(f"pin run broke (exit {p.returncode}):\n{p.stdout.decode()[-2000:]}")
    return p.returncode


def test_every_planted_mistake_fails_a_pin(tmp_path):
    text = SOURCE.read_text()
    jobs = []
    control_src, control_so = tmp_path / "control.c", tmp_path / "control.so"
    control_src.write_text(text)
    _compile(control_src, control_so)
    jobs.append(("unchanged source", control_src, control_so))
    for k, (name, old, new) in enumerate(MUTANTS):
        assert text.count(old) == 1, f"mutant {k} ({name}): the source no longer has this text exactly once"
        src, so = tmp_path / f"mutant{k}.c", tmp_path / f"mutant{k}.so"
        src.write_text(text.replace(old, new))
        _compile(src, so)
        jobs.append((name, src, so))
    workers = max(1, min(8, len(os.sched_getaffinity(0))))
    with ThreadPoolExecutor(max_workers=workers) as pool:
        codes = list(pool.map(lambda j: _run_battery(j[1], j[2]), jobs))
    assert codes[0] == 0, "the pins fail on the unchanged oracle"
    survivors = [name for (name, _, _), c in zip(jobs[1:], codes[1:]) if c == 0]
    assert not survivors, f"no pin noticed: {survivors}"


# The composite-drafting rule lives in the oracle's Python front end; same game there.  (No planted mistake hands a
# state of one automaton to another: that reads outside the arrays instead of giving a wrong answer.)
FRONT_END = ROOT / "oracle" / "__init__.py"
PY_MUTANTS = [
    ("the highest slot wins a tie",
     "if best_score is None or score > best_score:", "if best_score is None or score >= best_score:"),
    ("weights ignored",
     "score = np.float32(weights[b, m]) * np.float32(L)", "score = np.float32(L)"),
    ("match lengths ignored",
     "score = np.float32(weights[b, m]) * np.float32(L)", "score = np.float32(weights[b, m])"),
    ("a slot below min_match may still be chosen",
     "            if L < min_match:\n                continue\n", ""),
    ("a slot's matched length is not carried to the next call",
     "state[b, m], matched_len[b, m] = s, L", "state[b, m] = s"),
    ("an empty slot is not skipped",
     "            if slots[b, m] < 0:\n                continue\n", ""),
]

_PY_CHILD = r"""
import sys
sys.path.insert(0, {root!r})
sys.path.insert(0, {pkg_parent!r})          # the changed copy of the package shadows the real one
import oracle
assert oracle.__file__.startswith({pkg_parent!r})
import pytest
sys.exit(pytest.main(["-x", "-q", "-p", "no:cacheprovider", "tests/test_oracle_multi.py"]))
"""


def test_every_planted_mistake_in_the_composite_rule_fails_a_pin(tmp_path):
    text = FRONT_END.read_text()
    variants = [("unchanged source", text)]
    for k, (name, old, new) in enumerate(PY_MUTANTS):
        assert text.count(old) == 1, f"mutant {k} ({name}): the source no longer has this text exactly once"
        variants.append((name, text.replace(old, new)))

    def run(k):
        parent = tmp_path / f"pkg{k}"
        (parent / "oracle").mkdir(parents=True)
        (parent / "oracle" / "__init__.py").write_text(variants[k][1])
        (parent / "oracle" / "sam_oracle.c").write_text(SOURCE.read_text())
        code = _PY_CHILD.format(root=str(ROOT), pkg_parent=str(parent))
        p = subprocess.run([sys.executable, "-c", code], cwd=str(ROOT), env=dict(os.environ, OMP_NUM_THREADS="1"),
                           stdout=subprocess.PIPE, stderr=subprocess.STDOUT, timeout=600)
        if p.returncode not in (0, 1):
            raise RuntimeError(f"pin run broke (exit {p.returncode}):\n{p.stdout.decode()[-2000:]}")
        return p.returncode

    with ThreadPoolExecutor(max_workers=max(1, min(8, len(os.sched_getaffinity(0))))) as pool:
        codes = list(pool.map(run, range(len(variants))))
    assert codes[0] == 0, "the pins fail on the unchanged front end"
    survivors = [name for (name, _), c in zip(variants[1:], codes[1:]) if c == 0]
    assert not survivors, f"no pin noticed: {survivors}"
