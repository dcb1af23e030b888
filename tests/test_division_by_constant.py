"""The decode kernels divide a group's range by qmax = 3, 15 or 255 with a multiply and two fused
multiply-adds instead of a division (c = RN(1/qmax); q0 = RN(r c); rem = fma(-qmax, q0, r);
q = fma(rem, c, q0)).  The format defines scale = r / qmax in IEEE binary32, so the shortcut is only
admissible if it gives the same bits for every r it can meet: every binary32 value in
[2^-100, FLT_MAX] (smaller or overflowed ranges are stored flat).  That is 1.9e9 values per divisor,
few enough to try them all on the host cores in a few seconds."""
import subprocess

import pytest

SOURCE = r"""
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>
static inline float u2f(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }
static inline uint32_t f2u(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
int main(int argc, char **argv)
{
    const float ds[3] = {3.0f, 15.0f, 255.0f};
    const int broken = argc > 1;                       /* negative control: drop the correction step */
    const uint32_t lo = f2u(0x1p-100f), hi = f2u(3.402823466e+38f);
    for (int k = 0; k < 3; ++k) {
        const float d = ds[k], c = 1.0f / d;
        uint64_t bad = 0;
#pragma omp parallel for reduction(+ : bad)
        for (uint32_t u = lo; u <= hi; ++u) {
            const float r = u2f(u);
            const float q0 = r * c;
            const float rem = fmaf(-d, q0, r);
            const float q = broken ? q0 : fmaf(rem, c, q0);
            bad += f2u(q) != f2u(r / d);
        }
        printf("%g %llu %llu\n", d, (unsigned long long)(hi - lo) + 1, (unsigned long long)bad);
    }
    return 0;
}
"""


@pytest.fixture(scope="module")
def checker(tmp_path_factory):
    d = tmp_path_factory.mktemp("div")
    (d / "div.c").write_text(SOURCE)
    flags = ["-O3", "-ffp-contract=off", "-fopenmp"]
    if "fma" in open("/proc/cpuinfo").read():
        flags += ["-mfma", "-mavx2"]                    # fmaf() as one instruction; without it libm's exact fmaf runs
    subprocess.run(["gcc", *flags, "-o", str(d / "div"), str(d / "div.c"), "-lm"], check=True)
    return str(d / "div")


def test_three_instruction_division_equals_ieee_division_for_every_range(checker):
    out = subprocess.run([checker], check=True, capture_output=True, text=True, timeout=900).stdout.split("\n")
    rows = [ln.split() for ln in out if ln]
    assert [r[0] for r in rows] == ["3", "15", "255"]
    for d, n, bad in rows:
        assert int(n) == 1912602624 and int(bad) == 0, (d, n, bad)


def test_the_check_can_fail(checker):
    """Without the correction step a third or more of the quotients are off by an ulp."""
    out = subprocess.run([checker, "broken"], check=True, capture_output=True, text=True, timeout=900).stdout.split("\n")
    assert all(int(ln.split()[2]) > 10**8 for ln in out if ln)
