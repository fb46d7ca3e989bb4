"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's C
source (never in the GPU code), builds it, and runs the pin tests against that copy in a
child process: at least one pin must fail.  The unmodified copy must pass."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "wash_oracle.c")

MUTATIONS = {
    "philox multiplier": ("0xD2511F53u", "0xD2511F55u", "test_oracle_philox.py"),
    "weyl constant": ("k0 += 0x9E3779B9u;", "k0 += 0x9E3779B1u;", "test_oracle_philox.py"),
    "round drops a counter word": ("uint32_t n0 = hi1 ^ c1 ^ k0;", "uint32_t n0 = hi1 ^ k0;", "test_oracle_philox.py"),
    "output words swapped": ("out[0] = c0; out[1] = c1;", "out[0] = c1; out[1] = c0;", "test_oracle_philox.py"),
    "permutation stream shares the mask's tag": ("(uint32_t)((step >> 32) << 8) | (1u + block) };", "(uint32_t)((step >> 32) << 8) | (block) };", "test_oracle_philox.py"),
    "threshold off by one ulp of the word": ("floor(p * 4294967296.0)", "floor(p * 4294967295.0)", "test_oracle_philox.py"),
    "scatter instead of gather": ("a[wo_index(pop, n, elem)] = old[perm[n]];", "a[wo_index(pop, perm[n], elem)] = old[n];", "test_oracle_shuffle.py"),
    "never a fixed point (j below k)": ("* (uint64_t)(k + 1)) >> 32);", "* (uint64_t)(k)) >> 32);", "test_oracle_shuffle.py"),
    "mask decision inverted": ("if ((uint64_t)w >= thr) continue;", "if ((uint64_t)w < thr) continue;", "test_oracle_shuffle.py"),
    "second stack not permuted": ("if (stack2) wo_permute_column(pop, stack2, dtype2, pop->offset[s] + c, perm);", "", "test_oracle_shuffle.py"),
    "moved counts every value": ("moved += (perm[n] != n);", "moved += 1;", "test_oracle_shuffle.py"),
    "slice ignores its first coordinate": ("const uint64_t i = (uint64_t)(i0 + c);", "const uint64_t i = (uint64_t)(c);", "test_oracle_shuffle.py"),
    "ema weights swapped": ("float keep = alpha * wo_load(stack, dtype, idx);", "float keep = one_minus_alpha * wo_load(stack, dtype, idx);", "test_oracle_ema_avg.py"),
    "mean over N-1": ("float m = s / (float)pop->N;", "float m = s / (float)(pop->N - 1);", "test_oracle_ema_avg.py"),
    "sum from the last model down": ("for (int n = 1; n < pop->N; ++n) {\n        float x = wo_load(stack, dtype, wo_index(pop, n, elem));",
                                       "for (int n = pop->N - 1; n >= 1; --n) {\n        float x = wo_load(stack, dtype, wo_index(pop, n, elem));", "test_oracle_ema_avg.py"),
    "bf16 truncates": ("u += 0x7FFFu + lsb;", "", "test_oracle_ema_avg.py"),
    "worker sends along the inverse permutation": ("if (perm[n] != self) continue;", "if (perm[self] != n) continue;", "test_oracle_exchange.py"),
    "fixed points take a slot": ("if (perm[n] == n) continue;              /* worker n keeps its own value     */", "", "test_oracle_exchange.py"),
    "receiver takes a slot for a fixed point": ("if (perm[self] == self) continue;", "", "test_oracle_exchange.py"),
    "slot counts include fixed points": ("need[n] += (perm[n] != n);", "need[n] += 1;", "test_oracle_exchange.py"),
    "slots numbered per sender": ("const int64_t slot = next[n]++;\n                if (perm[n] != self) continue;           /* another worker fills this slot   */",
                                  "if (perm[n] != self) continue;\n                const int64_t slot = next[n]++;", "test_oracle_exchange.py"),
    "consensus sum lands in the next model's slot": ("sq_out[n] += dlt * dlt;", "sq_out[(n + 1) % pop->N] += dlt * dlt;", "test_oracle_ema_avg.py"),
    "consensus ignores the first tensor of its range": ("for (int s = seg_lo; s < seg_hi; ++s) {\n        for (int64_t c = 0; c < pop->numel[s]; ++c) {\n            int64_t elem = pop->offset[s] + c;\n            double mean = 0.0;",
                                                        "for (int s = 0; s < seg_hi; ++s) {\n        for (int64_t c = 0; c < pop->numel[s]; ++c) {\n            int64_t elem = pop->offset[s] + c;\n            double mean = 0.0;", "test_oracle_ema_avg.py"),
    "consensus divides the mean by N-1": ("mean /= (double)pop->N;", "mean /= (double)(pop->N - 1);", "test_oracle_ema_avg.py"),
    "last layer still shuffled": ("(double)l / (double)(L - 1);", "(double)l / (double)(L);", "test_oracle_ema_avg.py"),
}


def _build(text, path):
    src = path + ".c"
    with open(src, "w") as f:
        f.write(text)
    subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
                    "-o", path, src, "-lm"], check=True)


def _pins_pass(lib, test_file):
    env = dict(os.environ, WASH_ORACLE_LIB=lib)
    res = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                          os.path.join(ROOT, "tests", test_file)], env=env, cwd=ROOT, capture_output=True, text=True)
    return res.returncode == 0, res.stdout[-600:]


def test_unmodified_copy_passes_the_pins(tmp_path):
    with open(SRC) as f:
        text = f.read()
    lib = str(tmp_path / "liboracle_copy.so")
    _build(text, lib)
    for test_file in ("test_oracle_philox.py", "test_oracle_shuffle.py", "test_oracle_ema_avg.py", "test_oracle_exchange.py"):
        ok, tail = _pins_pass(lib, test_file)
        assert ok, tail


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_a_planted_mistake_is_caught(name, tmp_path):
    old, new, test_file = MUTATIONS[name]
    with open(SRC) as f:
        text = f.read()
    assert text.count(old) >= 1, "mutation target not found: %r" % old
    lib = str(tmp_path / "liboracle_mutant.so")
    _build(text.replace(old, new), lib)
    ok, tail = _pins_pass(lib, test_file)
    assert not ok, "no pin noticed the mistake %r\n%s" % (name, tail)
