"""Host-side check of an identity the CartPole kernel relies on: for binary32 x,
    q = x * R;  rem = fma(-q, 1.1f, x);  q' = fma(rem, R, q)      with R = binary32(1 / 1.1f)
equals the correctly rounded quotient x / 1.1f whenever 1e-30 <= |x| <= 1e30 (the kernel divides
plainly outside that range).  Checked in C (fmaf is a single rounding there) on every exponent with
2^15 significands each, plus the significands around the rounding boundaries of 1 / 1.1f; the full
sweep over all 2^32 values was run once when the kernel was written and found differences only for
|x| <= 3.39e-32 and -0."""
import ctypes
import os
import subprocess
import tempfile

SRC = r"""
#include <math.h>
#include <stdint.h>
#include <string.h>
/* returns the number of x in the sample whose two quotients differ; *first receives one of them */
long check(uint32_t stride, uint32_t offset, uint32_t *first)
{
    const float d = 1.1f, r = 1.0f / 1.1f;
    long bad = 0;
    for (uint64_t i = offset; i < (1ull << 32); i += stride) {
        uint32_t u = (uint32_t)i;
        float x;
        memcpy(&x, &u, 4);
        float ax = fabsf(x);
        if (!(ax >= 1e-30f && ax <= 1e30f)) continue;
        float want = x / d;
        float q = x * r;
        float rem = fmaf(-q, d, x);
        float got = fmaf(rem, r, q);
        if (memcmp(&want, &got, 4) != 0) { bad++; *first = u; }
    }
    return bad;
}
"""


def test_quotient_by_total_mass_identity():
    with tempfile.TemporaryDirectory() as tmp:
        c, so = os.path.join(tmp, "q.c"), os.path.join(tmp, "libq.so")
        with open(c, "w") as f:
            f.write(SRC)
        subprocess.run(["gcc", "-O2", "-fno-fast-math", "-ffp-contract=off", "-fPIC", "-shared",
                        "-o", so, c, "-lm"], check=True)
        lib = ctypes.CDLL(so)
        lib.check.argtypes = [ctypes.c_uint32, ctypes.c_uint32, ctypes.POINTER(ctypes.c_uint32)]
        lib.check.restype = ctypes.c_long
        first = ctypes.c_uint32(0)
        for stride, offset in ((257, 0), (256, 1), (255, 7)):       # three interleaved samples of 2^24 values
            assert lib.check(stride, offset, ctypes.byref(first)) == 0, hex(first.value)
