// Plan-time construction of the small Hadamard factor H_m (host code).
//
// Algorithm 2 of the paper builds a Hadamard matrix of order p + 1 from the Legendre symbols of
// a prime p = 3 (mod 4) (Section 2.3.3): H[0][0] = +1, the rest of the first row and column and
// the diagonal are -1, and H[i][j] = chi((i-1) - (j-1)) elsewhere.  Order 28 (needed for width
// 3584 = 28 * 128) has p = 27 = 3^3, so the same algorithm is run over the field GF(27) with chi
// its quadratic character; elements are indexed e = c0 + 3 c1 + 9 c2 for c0 + c1 x + c2 x^2 in
// GF(3)[x] / (x^3 + 2x + 1).
#include "gbs_internal.h"

namespace {

// Euler's criterion: chi(a) = a^((p-1)/2) mod p, mapped to {0, +1, -1}.
int chi_prime(int a, int p)
{
    a %= p;
    if (a < 0) a += p;
    if (a == 0) return 0;
    long long base = a, acc = 1;
    for (int e = (p - 1) / 2; e > 0; e >>= 1) {
        if (e & 1) acc = (acc * base) % p;
        base = (base * base) % p;
    }
    return acc == 1 ? +1 : -1;
}

bool prime_3_mod_4(int p)
{
    if (p < 3 || p % 4 != 3) return false;
    for (int q = 2; q * q <= p; ++q)
        if (p % q == 0) return false;
    return true;
}

// GF(27): multiply an element by x.  (c0, c1, c2) -> x*(c0 + c1 x + c2 x^2)
//   = c0 x + c1 x^2 + c2 x^3,  x^3 = -2x - 1 = x + 2  (mod 3)
int gf27_times_x(int e)
{
    int c0 = e % 3, c1 = (e / 3) % 3, c2 = e / 9;
    int n0 = (2 * c2) % 3;
    int n1 = (c0 + c2) % 3;
    int n2 = c1;
    return n0 + 3 * n1 + 9 * n2;
}

// chi over GF(27) from discrete logarithms to the base x (x is primitive: order 26):
// the non-zero squares are exactly the even powers.
void chi_gf27(int chi[27])
{
    chi[0] = 0;
    int e = 1;                                  // x^0
    for (int t = 0; t < 26; ++t) {
        chi[e] = (t % 2 == 0) ? +1 : -1;
        e = gf27_times_x(e);
    }
}

int gf27_minus(int e, int f)
{
    int r = 0, w = 1;
    for (int t = 0; t < 3; ++t, w *= 3) {
        int a = (e / w) % 3, b = (f / w) % 3;
        r += w * ((a + 3 - b) % 3);
    }
    return r;
}

}  // namespace

// Orders with a construction here: 1 (no Paley factor), p + 1 for the primes p = 3 (mod 4) up to 107
// that are multiples of 4 not covered by a smaller factor times a power of two, and 28 = 27 + 1.
bool gbs_supported_m(int m)
{
    static const int orders[] = {1, 12, 20, 24, 28, 44, 48, 60, 68, 72, 80, 84, 104, 108};
    for (int o : orders)
        if (m == o) return true;
    return false;
}

// Full orders (the whole rotation is H_m, Section 5.2.2): p = m - 1 prime, p = 3 (mod 4), m a multiple of 8 so that
// packed rows are whole bytes, large enough to be worth a dense tensor-core contraction and small enough for its image.
bool gbs_supported_full_m(int m)
{
    return m >= 128 && m <= 4096 && m % 8 == 0 && prime_3_mod_4(m - 1);
}

int gbs_build_hadamard_m(int m, int8_t* H)
{
    if (m == 1) { H[0] = 1; return GBS_OK; }
    int chi27[27];
    const bool field = (m == 28);
    if (field) chi_gf27(chi27);
    else if (!prime_3_mod_4(m - 1)) return GBS_ERR_UNSUPPORTED;
    for (int i = 0; i < m; ++i)
        for (int j = 0; j < m; ++j) {
            int v;
            if (i == 0 && j == 0) v = 1;
            else if (i == 0 || j == 0 || i == j) v = -1;
            else v = field ? chi27[gf27_minus(i - 1, j - 1)] : chi_prime((i - 1) - (j - 1), m - 1);
            H[i * m + j] = (int8_t)v;
        }
    return GBS_OK;
}
