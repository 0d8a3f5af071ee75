/* Host check behind the one-correction quotient of the CUDA kernels (not part of the oracle, shares
 * nothing with it): q1 = RN(q0 - r R), q0 = RN(a R), r = RN(q0 b - a), R = RN(1 / b) must equal the
 * IEEE quotient RN(a / b) for every pair of binary32 numbers.
 *
 * The value that the last FMA rounds differs from a / b by at most 3.5 * 2^-48 (for a quotient
 * scaled into [1/2, 2)), so q1 can be wrong only when a / b lies that close to the midpoint M of two
 * neighbouring floats.  With a = A 2^-23, b = B 2^-23 (A, B in [2^23, 2^24)):
 *   quotient in [1, 2):    M = m 2^-24, m odd in [2^24, 2^25):  a - b M = (A 2^24 - B m) 2^-47
 *   quotient in [1/2, 1):  M = m 2^-25, m odd in [2^24, 2^25):  a - b M = (A 2^25 - B m) 2^-48
 * and "that close" means |A 2^K - B m| <= 6.  This program enumerates every (A, B) with
 * |A 2^K - B m| <= 16 for some odd m, evaluates the kernel's arithmetic (both sign arrangements
 * used in the kernels) and the IEEE division in binary32, and counts the disagreements.  It also
 * counts how often the uncorrected q0 is wrong on the same pairs, to show that the pairs are hard.
 * Build: gcc -O2 -ffp-contract=off.  Prints "tested T failures F uncorrected_wrong U". */
#include <math.h>
#include <stdint.h>
#include <stdio.h>

#define NMAX 16

static long tested = 0, failures = 0, uncorrected_wrong = 0;

static void test_pair(uint32_t A, uint32_t B)
{
    float a = (float)A * 0x1p-23f, b = (float)B * 0x1p-23f;
    float R = 1.0f / b, t = a / b;
    float q = a * R, r = fmaf(q, b, -a), q1 = fmaf(-r, R, q);
    /* the arrangement of the packed code: q = (-a)(-R), r = q b + (-a), q1 = q + r (-R) */
    float na = -a, nR = -R, q2 = na * nR, r2 = fmaf(q2, b, na), q3 = fmaf(r2, nR, q2);
    /* the arrangement of the search kernel: r = q (-b) + a, q1 = q + r R */
    float r4 = fmaf(q, -b, a), q5 = fmaf(r4, R, q);
    ++tested;
    if (q1 != t || q3 != t || q5 != t) ++failures;
    if (q != t) ++uncorrected_wrong;
}

/* inverse of an odd x modulo 2^64 (Newton iteration) */
static uint64_t inverse_mod_2_64(uint64_t x)
{
    uint64_t y = x;
    for (int i = 0; i < 6; ++i) y *= 2 - x * y;
    return y;
}

int main(void)
{
    for (int K = 24; K <= 25; ++K) {
        for (uint32_t B = 1u << 23; B < (1u << 24); ++B) {
            int j = __builtin_ctz(B); /* B = 2^j Bo with Bo odd */
            uint64_t inv = inverse_mod_2_64(B >> j);
            for (int N = -NMAX; N <= NMAX; ++N) {
                /* A 2^K - B m = N  <=>  B m = -N (mod 2^K); solvable only if 2^j divides N */
                if (N == 0 || j > 4 || N % (1 << j) != 0) continue;
                uint64_t mod2 = 1ull << (K - j);
                uint64_t m0 = ((uint64_t)(-(int64_t)N / (1 << j)) * inv) & (mod2 - 1);
                for (uint64_t m = m0; m < (1ull << 25); m += mod2) {
                    if (m < (1ull << 24) || !(m & 1)) continue;
                    __int128 num = (__int128)B * m + N;
                    if (num % ((__int128)1 << K) != 0) continue;
                    uint64_t A = (uint64_t)(num >> K);
                    if (A < (1u << 23) || A >= (1u << 24)) continue;
                    if ((K == 24) != (A >= B)) continue; /* K = 24: quotient in [1, 2); K = 25: in [1/2, 1) */
                    test_pair((uint32_t)A, B);
                }
            }
        }
    }
    printf("tested %ld failures %ld uncorrected_wrong %ld\n", tested, failures, uncorrected_wrong);
    return failures != 0;
}
