// Winograd generator (Eq. 8).  Toom-Cook with a point at infinity:
//   * the polynomial of Eq. 8, M(x) = prod_i (x - p_i), has the alpha-1 finite
//     interpolation points as its roots; the alpha-th point is infinity;
//   * a product s = g * u of a k-term and an m-term polynomial has alpha = m+k-1
//     coefficients and is recovered from its values at the points by
//       s(x) = s_inf M(x) + sum_i s(p_i) L_i(x) / N_i,
//       L_i(x) = prod_{j != i} (x - p_j),  N_i = L_i(p_i),  s_inf = g_{k-1} u_{m-1};
//   * transposing that factorisation of the Toeplitz matrix of g turns it into the
//     m-output correlation  y = A^T [ (G g) (.) (B^T d) ]  with
//       A  (alpha x m):  rows [1, p_i, ..., p_i^{m-1}], infinity row [0,..,0,1]
//       G  (alpha x k):  rows [1, p_i, ..., p_i^{k-1}] / N_i, infinity row [0,..,0,1]
//       B^T(alpha x alpha): row i = coefficients of L_i(x) (ascending powers),
//                           last row = coefficients of M(x).
#include "generator.h"

#include <cmath>
#include <cstdint>
#include <cstring>

namespace mnnb {

namespace {

__int128 abs128(__int128 v) { return v < 0 ? -v : v; }

__int128 gcd128(__int128 a, __int128 b)
{
    a = abs128(a);
    b = abs128(b);
    while (b != 0) {
        __int128 t = a % b;
        a = b;
        b = t;
    }
    return a;
}

Rational make_reduced(__int128 n, __int128 d)
{
    Rational r;
    if (d < 0) {
        n = -n;
        d = -d;
    }
    if (n == 0) {
        r.num = 0;
        r.den = 1;
        return r;
    }
    __int128 g = gcd128(n, d);
    r.num = n / g;
    r.den = d / g;
    return r;
}

}  // namespace

Rational::Rational(long long n, long long d)
{
    Rational r = make_reduced(n, d);
    num = r.num;
    den = r.den;
}
Rational Rational::operator+(const Rational& o) const { return make_reduced(num * o.den + o.num * den, den * o.den); }
Rational Rational::operator-(const Rational& o) const { return make_reduced(num * o.den - o.num * den, den * o.den); }
Rational Rational::operator*(const Rational& o) const { return make_reduced(num * o.num, den * o.den); }
Rational Rational::operator/(const Rational& o) const { return make_reduced(num * o.den, den * o.num); }
Rational Rational::operator-() const
{
    Rational r;
    r.num = -num;
    r.den = den;
    return r;
}

double Rational::to_double() const
{
    const __int128 lim = (__int128)1 << 53;
    if (abs128(num) < lim && den < lim) {
        // both exactly representable: IEEE division rounds the exact quotient once
        return (double)(long long)num / (double)(long long)den;
    }
    return (double)((long double)num / (long double)den);
}

float Rational::to_float() const
{
    if (num == 0) return 0.0f;
    const double d = to_double();
    float f = (float)d;
    // (float)(double) can round twice; choose among f and its neighbours by exact comparison
    // of |c - num/den| = |c_mant * 2^e * den - num| / den.
    float cand[3] = {std::nextafterf(f, -INFINITY), f, std::nextafterf(f, INFINITY)};
    int best = 1;
    __int128 best_err = -1;
    // Express every candidate at one common binary scale (the smallest exponent).
    int exps[3];
    long long mants[3];
    int min_sh = 1 << 30;
    for (int i = 0; i < 3; ++i) {
        int e;
        double mant = std::frexp((double)cand[i], &e);
        mants[i] = (long long)std::ldexp(mant, 24);
        exps[i] = e - 24;
        if (exps[i] < min_sh) min_sh = exps[i];
    }
    for (int i = 0; i < 3; ++i) {
        __int128 lhs = ((__int128)mants[i] << (exps[i] - min_sh)) * den;   // cand * 2^-min_sh * den
        __int128 rhs = num;
        if (min_sh > 40 || min_sh < -60) return f;          // outside the range the generator produces
        if (min_sh >= 0) lhs <<= min_sh; else rhs <<= (-min_sh);
        __int128 err = abs128(lhs - rhs);
        bool even = (mants[i] & 1) == 0;
        if (best_err < 0 || err < best_err) {
            best_err = err;
            best = i;
        } else if (err == best_err && even) {
            best = i;
        }
    }
    return cand[best];
}

bool interpolation_points(int alpha, int points_id, std::vector<Rational>* out)
{
    out->clear();
    const int need = alpha - 1;
    if (need < 0) return false;
    std::vector<Rational> seq;
    seq.push_back(Rational(0));
    if (points_id == 1 || points_id == 2) {
        const Rational f = points_id == 1 ? Rational(1, 2) : Rational(1);
        for (int j = 1; (int)seq.size() < need; ++j) {
            seq.push_back(Rational(j) * f);
            seq.push_back(-(Rational(j) * f));
        }
    } else if (points_id == 3) {
        const Rational mags[] = {Rational(1), Rational(1, 2), Rational(2), Rational(1, 4), Rational(4),
                                 Rational(3, 4), Rational(4, 3)};
        for (const Rational& v : mags) {
            seq.push_back(v);
            seq.push_back(-v);
        }
        if (need > (int)seq.size()) return false;
    } else {
        return false;
    }
    out->assign(seq.begin(), seq.begin() + need);
    return true;
}

static std::vector<Rational> poly_mul_linear(const std::vector<Rational>& a, const Rational& root)
{
    // a(x) * (x - root), ascending powers
    std::vector<Rational> r(a.size() + 1);
    for (size_t i = 0; i < a.size(); ++i) {
        r[i] = r[i] - a[i] * root;
        r[i + 1] = r[i + 1] + a[i];
    }
    return r;
}

bool generate_winograd(int m, int k, int points_id, WinogradMatrices* out)
{
    if (m < 1 || k < 1) return false;
    const int alpha = m + k - 1;
    if (alpha > kMaxAlpha) return false;
    std::vector<Rational> p;
    if (!interpolation_points(alpha, points_id, &p)) return false;

    out->m = m;
    out->k = k;
    out->alpha = alpha;
    out->points_id = points_id;
    out->At.assign((size_t)m * alpha, Rational(0));
    out->G.assign((size_t)alpha * k, Rational(0));
    out->Bt.assign((size_t)alpha * alpha, Rational(0));

    for (int i = 0; i < alpha - 1; ++i) {
        Rational Ni(1);
        std::vector<Rational> Li(1, Rational(1));
        for (int j = 0; j < alpha - 1; ++j) {
            if (j == i) continue;
            Ni = Ni * (p[i] - p[j]);
            Li = poly_mul_linear(Li, p[j]);
        }
        Rational pw(1);
        for (int j = 0; j < m; ++j) {
            out->At[(size_t)j * alpha + i] = pw;       // A[i][j] = p_i^j, stored transposed
            pw = pw * p[i];
        }
        pw = Rational(1);
        for (int j = 0; j < k; ++j) {
            out->G[(size_t)i * k + j] = pw / Ni;
            pw = pw * p[i];
        }
        for (size_t j = 0; j < Li.size(); ++j) out->Bt[(size_t)i * alpha + j] = Li[j];
    }
    std::vector<Rational> Mx(1, Rational(1));
    for (int j = 0; j < alpha - 1; ++j) Mx = poly_mul_linear(Mx, p[j]);
    out->At[(size_t)(m - 1) * alpha + (alpha - 1)] = Rational(1);
    out->G[(size_t)(alpha - 1) * k + (k - 1)] = Rational(1);
    for (size_t j = 0; j < Mx.size(); ++j) out->Bt[(size_t)(alpha - 1) * alpha + j] = Mx[j];

    auto round_all = [](const std::vector<Rational>& src, std::vector<float>* f32, std::vector<double>* f64) {
        f32->resize(src.size());
        f64->resize(src.size());
        for (size_t i = 0; i < src.size(); ++i) {
            (*f32)[i] = src[i].to_float();
            (*f64)[i] = src[i].to_double();
        }
    };
    round_all(out->At, &out->At32, &out->At64);
    round_all(out->G, &out->G32, &out->G64);
    round_all(out->Bt, &out->Bt32, &out->Bt64);
    return true;
}

}  // namespace mnnb
