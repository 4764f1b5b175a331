"""Do the oracle's pins have teeth?  Plausible mistakes are planted in a COPY
of the oracle's source, one at a time (a wrong sign, a swapped operand, a
dropped worker or term, eps inside the root, a missing bias correction, a
wrong half of the bf16 word, ...), the copy is compiled, and the pin files
are run against it in a child process: every one of them has to fail.  Each
mistake is planted in the binary32 AND the binary64 mode, so that the pin
"binary32 tracks binary64" cannot be what catches it: a closed form, a
hand-worked value or an invariant has to.

The mistakes live on the CPU, in the checker; nothing here touches the GPU.
"""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "ps_oracle.cpp")
PINS = ["tests/test_oracle_pins.py", "tests/test_oracle_ieee.py", "tests/test_oracle_service_pins.py"]

# name -> [(text in the oracle's source, replacement), ...]; every text must occur
MUTANTS = {
    "reduce: a worker subtracted": [
        ("G = G + shard_value(hp, k->shards[w], i);", "G = G - shard_value(hp, k->shards[w], i);"),
        ("G = G + (double)shard_value(hp, k->shards[w], i);", "G = G - (double)shard_value(hp, k->shards[w], i);")],
    "reduce: last worker dropped": [("for (int w = 1; w < W; ++w)", "for (int w = 1; w + 1 < W; ++w)")],
    "reduce: worker index off by one": [("k->shards[w], i)", "k->shards[w - 1], i)")],
    "reduce: mean instead of sum": [("G = G * gs;", "G = G * gs / W;")],
    "grad_scale dropped": [("G = G * gs;", "G = G * 1;")],
    "decay applied to the state": [("wd * p[i]", "wd * s0[i]")],
    "decay subtracted": [("const float d = G + wdp;", "const float d = G - wdp;"),
                         ("const double d = G + wd * p[i];", "const double d = G - wd * p[i];")],
    "decay dropped": [("const float d = G + wdp;", "const float d = G;"),
                      ("const double d = G + wd * p[i];", "const double d = G;")],
    "momentum taken from the parameter": [("mom * s0[i]", "mom * p[i]")],
    "velocity: gradient subtracted": [("const float v = mv + d;", "const float v = mv - d;"),
                                      ("const double v = mom * s0[i] + d;", "const double v = mom * s0[i] - d;")],
    "sgd: step from the gradient, not the velocity": [("const float step = lr * v;", "const float step = lr * d;"),
                                                       ("p[i] = p[i] - lr * v;", "p[i] = p[i] - lr * d;")],
    "sgd: lr inside the velocity": [("const float v = mv + d;", "const float v = mv + lr * d;"),
                                    ("const float step = lr * v;", "const float step = v;"),
                                    ("const double v = mom * s0[i] + d;", "const double v = mom * s0[i] + lr * d;"),
                                    ("p[i] = p[i] - lr * v;", "p[i] = p[i] - v;")],
    "ascent instead of descent": [("p[i] = p[i] - step;", "p[i] = p[i] + step;"),
                                  ("p[i] = p[i] - lr * v;", "p[i] = p[i] + lr * v;"),
                                  ("p[i] = p[i] - ss_t * (m / den);", "p[i] = p[i] + ss_t * (m / den);")],
    "sgd: velocity not stored": [("      s0[i] = v;\n", "      ;\n")],
    "adam: beta2 on the first moment": [("b1 * s0[i]", "b2 * s0[i]")],
    "adam: beta1 instead of 1 - beta1": [("omb1 * d", "b1 * d")],
    "adam: gradient not squared": [("const float dd = d * d;", "const float dd = d;"),
                                   ("omb2 * (d * d)", "omb2 * (d)")],
    "adam: beta1 on the second moment": [("b2 * s1[i]", "b1 * s1[i]")],
    "adam: beta2 instead of 1 - beta2": [("const float odd = omb2 * dd;", "const float odd = b2 * dd;"),
                                         ("omb2 * (d * d)", "b2 * (d * d)")],
    "adam: no square root": [("std::sqrt(v)", "(v)")],
    "adam: second bias correction multiplied": [("const float rh = r / sbc2_t;", "const float rh = r * sbc2_t;"),
                                                ("std::sqrt(v) / sbc2_t", "std::sqrt(v) * sbc2_t")],
    "adam: second bias correction dropped": [("const float rh = r / sbc2_t;", "const float rh = r;"),
                                             ("std::sqrt(v) / sbc2_t", "std::sqrt(v)")],
    "adam: eps dropped": [("const float den = rh + eps;", "const float den = rh;"),
                          ("/ sbc2_t + eps;", "/ sbc2_t;")],
    "adam: eps inside the root": [("const float r = std::sqrt(v);", "const float r = std::sqrt(v + eps);"),
                                  ("const float den = rh + eps;", "const float den = rh;"),
                                  ("const double den = std::sqrt(v) / sbc2_t + eps;",
                                   "const double den = std::sqrt(v + eps) / sbc2_t;")],
    "adam: quotient inverted": [("m / den", "den / m")],
    "adam: first bias correction dropped": [("(float)oracle_adam_step_size(lr, b1, k->step)", "lr"),
                                            ("= oracle_adam_step_size(hp->lr, hp->beta1, k->step)", "= lr")],
    "adam: first bias correction with the wrong sign": [
        ("(double)lr / (1.0 - std::pow((double)beta1, (double)t))", "(double)lr / (1.0 + std::pow((double)beta1, (double)t))")],
    "adam: first bias correction with beta^(t-1)": [
        ("(double)lr / (1.0 - std::pow((double)beta1, (double)t))", "(double)lr / (1.0 - std::pow((double)beta1, (double)t + 1.0))")],
    "adam: second bias correction without its root": [
        ("return std::sqrt(1.0 - std::pow((double)beta2, (double)t));", "return 1.0 - std::pow((double)beta2, (double)t);")],
    "adam: first moment not stored": [("      s0[i] = m;\n", "      ;\n")],
    "adam: second moment not stored": [("      s1[i] = v;\n", "      ;\n")],
    "adam: decay decoupled from the moments": [
        ("      const float q = m / den;\n      const float step = ss_t * q;",
         "      const float q = m / den;\n      const float step = ss_t * q + lr * wdp;"),
        ("const float od = omb1 * d;", "const float od = omb1 * G;"),
        ("const float dd = d * d;", "const float dd = G * G;"),
        ("const double m = b1 * s0[i] + omb1 * d;", "const double m = b1 * s0[i] + omb1 * G;"),
        ("const double v = b2 * s1[i] + omb2 * (d * d);", "const double v = b2 * s1[i] + omb2 * (G * G);"),
        ("p[i] = p[i] - ss_t * (m / den);", "p[i] = p[i] - ss_t * (m / den) - lr * wd * p[i];")],
    "norm: not squared": [("sq += (double)G * (double)G;", "sq += (double)G;"), ("sq += G * G;", "sq += G;")],
    "norm: taken before the scale": [("    G = G * gs;\n    sq += (double)G * (double)G;", "    sq += (double)G * (double)G;\n    G = G * gs;"),
                                     ("    G = G * gs;\n    sq += G * G;", "    sq += G * G;\n    G = G * gs;")],
    "blocks: the last task of a batch is skipped": [
        ("for (int b = 0; b < n; ++b) bad |= (oracle_block_step_f32(&tasks[b]) != 0);",
         "for (int b = 0; b < n - 1; ++b) bad |= (oracle_block_step_f32(&tasks[b]) != 0);")],
    "elements: the last element of a block is skipped": [("for (uint64_t i = 0; i < k->nelem; ++i) {", "for (uint64_t i = 0; i + 1 < k->nelem; ++i) {")],
    "bf16 array widening stops one short": [("for (uint64_t i = 0; i < n; ++i) out[i] = oracle_bf16_to_f32(bits[i]);",
                                             "for (uint64_t i = 0; i + 1 < n; ++i) out[i] = oracle_bf16_to_f32(bits[i]);")],
    "bf16: shifted by 15": [("(uint32_t)bits << 16", "(uint32_t)bits << 15")],
    "bf16: low half of the word": [("(uint32_t)bits << 16", "(uint32_t)bits")],
}


def _build(tmp, name, edits):
    src = open(SRC).read()
    for old, new in edits:
        assert src.count(old) >= 1, "mutant %r: text %r not in the oracle's source" % (name, old)
        src = src.replace(old, new)
    stem = "".join(c if c.isalnum() else "_" for c in name)
    cpp, lib = os.path.join(tmp, stem + ".cpp"), os.path.join(tmp, "lib" + stem + ".so")
    open(cpp, "w").write(src)
    subprocess.run(["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared",
                    "-w", "-o", lib, cpp], check=True)
    return lib


def _pins_pass(lib):
    """Runs the pin files in a child whose oracle loads `lib`; True if they all pass."""
    code = ("import sys; sys.path.insert(0, %r); import oracle.build as ob; ob.build = lambda force=False: %r; "
            "import pytest; sys.exit(pytest.main(['-x', '-q', '-p', 'no:cacheprovider'] + %r))" % (ROOT, lib, PINS))
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, capture_output=True, text=True,
                       env=dict(os.environ, OMP_NUM_THREADS="2"))
    assert r.returncode in (0, 1), "the pin run itself broke:\n" + r.stdout[-2000:] + r.stderr[-2000:]
    return r.returncode == 0


def test_every_planted_mistake_fails_a_pin(tmp_path):
    tmp = str(tmp_path)
    assert _pins_pass(_build(tmp, "control", [])), "the unchanged oracle must pass its pins"
    names = list(MUTANTS)
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        survived = [n for n, ok in zip(names, pool.map(lambda n: _pins_pass(_build(tmp, n, MUTANTS[n])), names)) if ok]
    assert not survived, "no pin notices: " + "; ".join(survived)
    assert len(names) >= 30


# ---------------------------------------------------------------- the assignment oracle (Pseudocode 1)

ASSIGN_SRC = os.path.join(ROOT, "oracle", "assignment.py")
ASSIGN_MUTANTS = {
    "cycle: the shortest period instead of the longest": [
        ("return max((self.D[j] for j in js), default=0.0)", "return min((self.D[j] for j in js), default=0.0)")],
    "stretched duration: one slot too many": [("max(D_j, C / r)", "max(D_j, C / (r + 1))")],
    "loss relative to the profiled duration": [("return (d_j - D_j) / d_j", "return (d_j - D_j) / D_j")],
    "loss limit doubled": [(">= self.loss_limit", ">= 2 * self.loss_limit")],
    "estimated cycle ignores the new job": [("C_est = max(self.cycle(n), self.D[k])", "C_est = max(self.cycle(n), 0.0)")],
    "free slots: multiplicity dropped": [
        ("free -= floor_ratio(C_est, d_j) * sum(self.N[n].tasks.get(j, {}).values())",
         "free -= sum(self.N[n].tasks.get(j, {}).values())")],
    "needed slots: multiplicity dropped": [
        ("need = floor_ratio(C_est, stretched_duration(self.D[k], C_est)) * e_t", "need = e_t")],
    "worst fit": [("F < best[1]", "F > best[1]")],
    "first fit": [("(best is None or F < best[1])", "best is None")],
    "any Aggregator with a free slot fits": [("F >= need - 1e-12", "F > 0")],
    "the new task's own job is not examined": [("sorted(set(self.N[n].jobs()) | {k})", "sorted(set(self.N[n].jobs()))")],
    "recycling starts from the heaviest": [("n = min(live, key=lambda i: (self.load(i), i))", "n = max(live, key=lambda i: (self.load(i), i))")],
    "recycling may re-place onto the same Aggregator": [("allow_new=False, exclude=n", "allow_new=False, exclude=-1")],
    "outlier: scheduled requests not reserved": [
        ("return (C_n - now_in_cycle) - remaining_scheduled >= e_late - 1e-12", "return (C_n - now_in_cycle) >= e_late - 1e-12")],
    "floor without its guard": [("int(math.floor(a / b * (1.0 + 1e-9) + 1e-12))", "int(math.floor(a / b))")],
    "load: multiplicity dropped": [("tot += floor_ratio(C, d) * sum(self.N[n].tasks[j].values())", "tot += sum(self.N[n].tasks[j].values())")],
    "empty Aggregators are not released": [("            if a.alive and not a.jobs():\n                a.alive = False\n                released += 1",
                                            "            if False:\n                a.alive = False\n                released += 1")],
}


def _assignment_pins_pass(tmp, name, edits):
    src = open(ASSIGN_SRC).read()
    for old, new in edits:
        assert src.count(old) >= 1, "mutant %r: text %r not in the assignment oracle" % (name, old)
        src = src.replace(old, new)
    path = os.path.join(tmp, "assignment_" + "".join(c if c.isalnum() else "_" for c in name) + ".py")
    open(path, "w").write(src)
    # the child loads the changed file as oracle.assignment, then runs the oracle's own pins
    # (the planner-parity tests need the library and are not what is being examined here)
    code = ("import sys, importlib.util; sys.path.insert(0, %r); import oracle; "
            "spec = importlib.util.spec_from_file_location('oracle.assignment', %r); m = importlib.util.module_from_spec(spec); "
            "sys.modules['oracle.assignment'] = m; spec.loader.exec_module(m); oracle.assignment = m; "
            "import pytest; sys.exit(pytest.main(['-x', '-q', '-p', 'no:cacheprovider', '-k', 'not planner', 'tests/test_assignment.py']))"
            % (ROOT, path))
    try:
        r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, capture_output=True, text=True, timeout=120)
    except subprocess.TimeoutExpired:
        return False                     # a mistake that never terminates is noticed too
    assert r.returncode in (0, 1), "the pin run itself broke:\n" + r.stdout[-2000:] + r.stderr[-2000:]
    return r.returncode == 0


def test_every_mistake_planted_in_the_assignment_oracle_fails_a_pin(tmp_path):
    tmp = str(tmp_path)
    assert _assignment_pins_pass(tmp, "control", []), "the unchanged assignment oracle must pass its pins"
    names = list(ASSIGN_MUTANTS)
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        survived = [n for n, ok in zip(names, pool.map(lambda n: _assignment_pins_pass(tmp, n, ASSIGN_MUTANTS[n]), names)) if ok]
    assert not survived, "no pin notices: " + "; ".join(survived)


# ---------------------------------------------------------------- the oracle's service semantics (Python)

SERVICE_SRC = os.path.join(ROOT, "oracle", "aggregator.py")
SERVICE_PINS = ["tests/test_oracle_pins.py", "tests/test_oracle_service_pins.py", "tests/test_rows.py"]
SERVICE_MUTANTS = {
    "step counter does not advance": [("            b.step += 1\n", "            b.step += 0\n")],
    "shards summed in arrival order, not worker order": [
        ("[b.pushed[w] for w in range(hp.num_workers)]", "list(b.pushed.values())")],
    "pushes not cleared by an aggregate": [("                b.pushed = {}\n", "                pass\n")],
    "a worker may push twice": [("        if worker in b.pushed:\n            raise ValueError(\"duplicate push\")", "        if False:\n            raise ValueError(\"duplicate push\")")],
    "a task that is not ready is skipped, not refused": [("                raise RuntimeError(\"not ready\")", "                continue")],
    "a task may be listed twice": [("            if key in seen:\n                raise ValueError(\"task listed twice\")", "            if False:\n                raise ValueError(\"task listed twice\")")],
    "unlisted rows are -0.0": [("        dense = np.zeros((b.nelem // row_len, row_len), dtype=_grad_np_dtype(hp))",
                                "        dense = -np.zeros((b.nelem // row_len, row_len), dtype=_grad_np_dtype(hp)) if _grad_np_dtype(hp) == np.float32 else np.zeros((b.nelem // row_len, row_len), dtype=np.uint16)")],
    "row ids may repeat": [("np.any(np.diff(ids) <= 0)", "np.any(np.diff(ids) < 0)")],
    "migration forgets the context": [("        b.ctx = dst_ctx\n", "        pass\n")],
    "migration restarts the step counter": [("        b.ctx = dst_ctx\n", "        b.ctx = dst_ctx\n        b.step = 0\n")],
    "migration drops the optimizer state": [("        b.p, b.s0 = b.p.copy(), b.s0.copy()", "        b.p, b.s0 = b.p.copy(), np.zeros_like(b.s0)")],
    "state does not start at zero": [("        s0 = np.zeros(nelem, np.float32)\n", "        s0 = np.ones(nelem, np.float32)\n")],
    "norms accumulate over iterations": [("                b.sqnorm = s\n", "                b.sqnorm += s\n")],
}


def _service_pins_pass(tmp, name, edits):
    src = open(SERVICE_SRC).read()
    for old, new in edits:
        assert src.count(old) >= 1, "mutant %r: text %r not in the oracle's service code" % (name, old)
        src = src.replace(old, new)
    path = os.path.join(tmp, "aggregator_" + "".join(c if c.isalnum() else "_" for c in name) + ".py")
    open(path, "w").write(src)
    code = ("import sys, importlib.util; sys.path.insert(0, %r); import oracle; "
            "spec = importlib.util.spec_from_file_location('oracle.aggregator', %r); m = importlib.util.module_from_spec(spec); "
            "sys.modules['oracle.aggregator'] = m; spec.loader.exec_module(m); oracle.aggregator = m; "
            "import pytest; sys.exit(pytest.main(['-x', '-q', '-p', 'no:cacheprovider', '-m', 'not gpu'] + %r))"
            % (ROOT, path, SERVICE_PINS))
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, capture_output=True, text=True, timeout=300,
                       env=dict(os.environ, OMP_NUM_THREADS="2"))
    assert r.returncode in (0, 1), "the pin run itself broke:\n" + r.stdout[-2000:] + r.stderr[-2000:]
    return r.returncode == 0


def test_every_mistake_planted_in_the_oracles_service_semantics_fails_a_pin(tmp_path):
    tmp = str(tmp_path)
    assert _service_pins_pass(tmp, "control", []), "the unchanged oracle must pass its pins"
    names = list(SERVICE_MUTANTS)
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        survived = [n for n, ok in zip(names, pool.map(lambda n: _service_pins_pass(tmp, n, SERVICE_MUTANTS[n]), names)) if ok]
    assert not survived, "no pin notices: " + "; ".join(survived)
