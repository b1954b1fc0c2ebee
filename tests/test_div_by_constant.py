"""The scale formulas of the double-block quantizer (paper Sec. 2.2) divide by two constants: S_global = amax / 2688 and
s = t / 6. The contract pins both as IEEE binary32 divisions; the CUDA kernels compute them as

    q0 = RN(x * rc),  rem = fma(-q0, c, x),  q = fma(rem, rc, q0),     rc = RN(1 / c)

(three instructions instead of a division routine). This test is the proof that the substitution changes nothing: the
sequence, restated here in C with the same two reciprocal constants, is compared with the correctly rounded quotient x / c
for EVERY non-negative finite binary32 x (2^31 - 2^23 values per constant). They must agree whenever the quotient is a normal
number; where they differ the quotient is subnormal, which for s = t / 6 is far below the smallest E4M3 value (both encode
to 0) and for S_global = amax / 2688 means amax < 2^-114, outside the supported range of inputs."""
import os
import subprocess
import sys

SRC = r"""
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>
static inline float u2f(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }
static inline uint32_t f2u(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
int main(void) {
  const float cs[2] = {6.0f, 2688.0f};
  const float rcs[2] = {0x1.555556p-3f, 0x1.861862p-12f};  /* the constants the kernels use */
  for (int ci = 0; ci < 2; ++ci) {
    const float c = cs[ci], rc = rcs[ci];
    if (f2u(rc) != f2u(1.0f / c)) { printf("rc of %g is not RN(1/c)\n", c); return 1; }
    long long differ = 0, differ_normal = 0;
    float largest_differing = 0.0f;
#pragma omp parallel for reduction(+ : differ, differ_normal) reduction(max : largest_differing) schedule(static)
    for (long long i = 0; i < 0x7F800000LL; ++i) {
      const float x = u2f((uint32_t)i);
      const float want = x / c;
      const float q0 = x * rc;
      const float rem = fmaf(-q0, c, x);
      const float q = fmaf(rem, rc, q0);
      if (f2u(q) != f2u(want)) {
        ++differ;
        if (want >= 1.17549435e-38f) ++differ_normal;
        if (want > largest_differing) largest_differing = want;
      }
    }
    printf("%g %lld %lld %a\n", c, differ, differ_normal, largest_differing);
  }
  return 0;
}
"""


def test_three_instruction_division_equals_the_ieee_quotient_for_every_input(tmp_path):
    src = tmp_path / "divcheck.c"
    exe = tmp_path / "divcheck"
    src.write_text(SRC)
    subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-mfma", str(src), "-o", str(exe), "-lm"])
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True, timeout=900).stdout.strip().splitlines()
    assert len(out) == 2, out
    for line, c in zip(out, (6.0, 2688.0)):
        cc, differ, differ_normal, largest = line.split()
        assert float(cc) == c
        assert int(differ_normal) == 0, line  # identical for every input whose quotient is a normal number
        assert float.fromhex(largest) < 2.0 ** -126, line  # the remaining differences are subnormal quotients
