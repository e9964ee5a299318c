"""Do the pins bite?  Mistakes are planted in COPIES of the oracle source (on the CPU, in a
temporary directory), each copy is compiled, and the pin suite must fail on every one of
them.  A plausible slip anywhere in the oracle -- a dropped term, a wrong sign, index or
operand -- has to be caught by at least one pin."""
import os
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

ENTROPY = "ecq_entropy_oracle.cpp"
SOURCES = ("ecq_oracle.cpp", ENTROPY)
PINS = {"ecq_oracle.cpp": "test_oracle_pins.py", ENTROPY: "test_oracle_entropy.py"}

# (what is planted, text to replace, replacement[, source file])
MUTATIONS = [
    ("compensation dropped (Eq. 7)", "v[i - lo] = std::fmaf(alpha, h[i], g[i]);", "v[i - lo] = g[i];"),
    ("compensation sign (Eq. 7)", "v[i - lo] = std::fmaf(alpha, h[i], g[i]);", "v[i - lo] = std::fmaf(-alpha, h[i], g[i]);"),
    ("round up with probability 1 - f (Eq. 9)", "const int32_t m = l + ((u < f) ? 1 : 0);", "const int32_t m = l + ((u < 1.0f - f) ? 1 : 0);"),
    ("never round up (Eq. 9)", "const int32_t m = l + ((u < f) ? 1 : 0);", "const int32_t m = l;"),
    ("sign of the level lost (Eq. 8)", "const int32_t q = (f2u(vi) >> 31) ? -m : m;", "const int32_t q = m;"),
    ("error update books +g~ (Eq. 6)", "const float e = ((mode == 0) ? g[i] : vi) - gq;", "const float e = ((mode == 0) ? g[i] : vi) + gq;"),
    ("error update books the compensated value (Eq. 6)", "const float e = ((mode == 0) ? g[i] : vi) - gq;", "const float e = vi - gq;"),
    ("decay dropped (Eq. 6)", "h[i] = std::fmaf(beta, h[i], e);\n        }\n        scales[b] = scale;", "h[i] = h[i] + e;\n        }\n        scales[b] = scale;"),
    ("level step scale/(s+1)", "a_step = scale / sf;", "a_step = scale / (sf + 1.0f);"),
    ("code width off by one", "while ((1ull << r) < 2ull * s + 1ull) ++r;", "while ((1ull << r) < 2ull * s) ++r;"),
    ("bit order within a code", "if ((c >> j) & 1u) words[k >> 5] |= (1u << (k & 31));", "if ((c >> (r - 1 - j)) & 1u) words[k >> 5] |= (1u << (k & 31));"),
    ("Philox multipliers swapped", "const uint64_t p0 = (uint64_t)kM0 * c0;", "const uint64_t p0 = (uint64_t)kM1 * c0;"),
    ("Philox counter: worker and step swapped", "{(uint32_t)blk, (uint32_t)(blk >> 32), worker, step}", "{(uint32_t)blk, (uint32_t)(blk >> 32), step, worker}"),
    ("Philox word of the next entry", "return out[i & 3];", "return out[(i + 1) & 3];"),
    ("draw uses the low 24 bits", "(float)(R >> 8) * 0x1p-24f", "(float)(R & 0xFFFFFFu) * 0x1p-24f"),
    ("scale is the max of v, not of |v|", "const uint32_t a = f2u(v[i - lo]) & 0x7FFFFFFFu;", "const uint32_t a = (f2u(v[i - lo]) >> 31) ? 0u : f2u(v[i - lo]);"),
    ("mean divides by W + 1 (Eq. 4)", "out[i] = acc / (float)W;", "out[i] = acc / (float)(W + 1);"),
    ("decode forgets the offset s", "(int32_t)get_code(codes[w], i * r, r) - (int32_t)s;\n            acc", "(int32_t)get_code(codes[w], i * r, r);\n            acc"),
    ("decode uses worker 0's scale for everyone", "const float a = scales[w][b] / sf;", "const float a = scales[0][b] / sf;"),
    ("update adds instead of subtracting (Algorithm 1)", "params[i] = std::fmaf(-eta, mean[i], params[i]);", "params[i] = std::fmaf(eta, mean[i], params[i]);"),
    ("l2 scale without the square root", "scale = std::sqrt(runs[0]);", "scale = runs[0];"),
    ("l2 runs summed back to front", "for (uint64_t j = i; j < hi && j < i + 32; ++j) acc = std::fmaf(v[j - lo], v[j - lo], acc);",
     "for (uint64_t j = (hi < i + 32 ? hi : i + 32); j-- > i;) acc = std::fmaf(v[j - lo], v[j - lo], acc);"),
    ("entropy bound in nats", "bits += (double)counts[k] * std::log2(d / (double)counts[k]);", "bits += (double)counts[k] * std::log(d / (double)counts[k]);"),
    ("zero bucket forgets the decay", "const float e = (mode == 0) ? g[i] : vi;\n                h[i] = std::fmaf(beta, h[i], e);", "const float e = (mode == 0) ? g[i] : vi;\n                h[i] = h[i] + e;"),
    ("package-merge takes one node too many", "for (size_t i = 0; i < 2 * n - 2; ++i) count_leaves", "for (size_t i = 0; i < 2 * n - 1; ++i) count_leaves", ENTROPY),
    ("package-merge merges without the leaves", "const std::vector<int32_t> leaves = new_leaves();", "const std::vector<int32_t> leaves;", ENTROPY),
    ("package-merge builds one level too few", "for (uint32_t level = 1; level < max_len; ++level) {", "for (uint32_t level = 2; level < max_len; ++level) {", ENTROPY),
    ("package-merge builds one level too many", "for (uint32_t level = 1; level < max_len; ++level) {", "for (uint32_t level = 0; level < max_len; ++level) {", ENTROPY),
    ("packages overlap", "for (size_t i = 0; i + 1 < list.size(); i += 2) {", "for (size_t i = 0; i + 1 < list.size(); i += 1) {", ENTROPY),
    ("canonical step adds after the shift", "if (i > 0) next = (next + 1) << (L - prev_len);", "if (i > 0) next = (next << (L - prev_len)) + 1;", ENTROPY),
    ("word sent last bit first", "const uint32_t b = (word[sym] >> (L - 1 - k)) & 1u;", "const uint32_t b = (word[sym] >> k) & 1u;", ENTROPY),
    ("chunks not aligned to words", "at = (bit + 31) / 32;\n    }\n    if (at > 0xFFFFFFFFull)", "at = bit / 32;\n    }\n    if (at > 0xFFFFFFFFull)", ENTROPY),
    ("chunk of 1000 entries", "const uint32_t kChunk = 1024;", "const uint32_t kChunk = 1000;", ENTROPY),
    ("quarter marks one entry late", "if (i > lo && (i - lo) % kQuarter == 0)\n                quarters[3 * c + (i - lo) / kQuarter - 1] = (uint16_t)(bit - at * 32);\n            const uint32_t sym = get_bits(codes, i * r, r);", "const uint32_t sym = get_bits(codes, i * r, r);\n            if (i > lo && (i - lo) % kQuarter == 0)\n                quarters[3 * c + (i - lo) / kQuarter - 1] = (uint16_t)(bit - at * 32 + lengths[sym < n_sym ? sym : 0]);", ENTROPY),
    ("quarter of 128 entries", "const uint32_t kQuarter = 256;", "const uint32_t kQuarter = 128;", ENTROPY),
    ("decoder reads the stream from bit 1", "uint64_t bit = (uint64_t)offsets[c] * 32;\n        for (uint64_t i = lo; i < hi; ++i) {\n            if (i > lo && (i - lo) % kQuarter == 0)\n                bit =", "uint64_t bit = (uint64_t)offsets[c] * 32 + 1;\n        for (uint64_t i = lo; i < hi; ++i) {\n            if (i > lo && (i - lo) % kQuarter == 0)\n                bit =", ENTROPY),
]


def _run_pins(oracle_dir, pins):
    env = dict(os.environ)
    env["PYTHONPATH"] = os.path.dirname(oracle_dir) + os.pathsep + ROOT
    return subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider"] +
                          [os.path.join(ROOT, "tests", p) for p in pins],
                          env=env, cwd=os.path.dirname(oracle_dir), capture_output=True, text=True,
                          timeout=900)


def test_every_planted_mistake_fails_a_pin(tmp_path):
    srcs = {f: open(os.path.join(ROOT, "oracle", f)).read() for f in SOURCES}
    def attempt(item):
        k, mutation = item
        what, old, new = mutation[:3]
        target = mutation[3] if len(mutation) > 3 else "ecq_oracle.cpp"
        assert srcs[target].count(old) == 1, "mutation target not found exactly once: " + what
        odir = tmp_path / ("m%02d" % k) / "oracle"
        odir.mkdir(parents=True)
        shutil.copy(os.path.join(ROOT, "oracle", "__init__.py"), odir / "__init__.py")
        for f in SOURCES:
            (odir / f).write_text(srcs[f].replace(old, new) if f == target else srcs[f])
        return what if _run_pins(str(odir), [PINS[target]]).returncode == 0 else None

    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        survivors = [w for w in ex.map(attempt, list(enumerate(MUTATIONS))) if w]
    assert not survivors, "pins did not notice: " + "; ".join(survivors)


def test_the_unmutated_copy_passes(tmp_path):
    odir = tmp_path / "clean" / "oracle"
    odir.mkdir(parents=True)
    for f in ("__init__.py",) + SOURCES:
        shutil.copy(os.path.join(ROOT, "oracle", f), odir / f)
    res = _run_pins(str(odir), list(PINS.values()))
    assert res.returncode == 0, res.stdout[-2000:]
