// Winograd generator (Eq. 8): transform matrices of F(m, k) from interpolation
// points, in exact rational arithmetic on the host, rounded once to fp32/fp64.
#pragma once
#include <vector>

namespace mnnb {

constexpr int kMaxAlpha = 16;

// Exact rational on 128-bit integers, always reduced, denominator > 0.
struct Rational {
    __int128 num = 0;
    __int128 den = 1;
    Rational() = default;
    Rational(long long n) : num(n), den(1) {}
    Rational(long long n, long long d);
    Rational operator+(const Rational& o) const;
    Rational operator-(const Rational& o) const;
    Rational operator*(const Rational& o) const;
    Rational operator/(const Rational& o) const;
    Rational operator-() const;
    bool operator==(const Rational& o) const { return num == o.num && den == o.den; }
    bool is_zero() const { return num == 0; }
    double to_double() const;   // correctly rounded
    float to_float() const;     // correctly rounded (nearest, ties to even)
};

struct WinogradMatrices {
    int m = 0, k = 0, alpha = 0, points_id = 0;
    // row-major: At [m][alpha], G [alpha][k], Bt [alpha][alpha]
    std::vector<Rational> At, G, Bt;
    std::vector<float> At32, G32, Bt32;
    std::vector<double> At64, G64, Bt64;
};

// The alpha-1 finite points of point set `points_id` (1 paper f=1/2, 2 unit, 3 mixed).
// Returns false if the set cannot supply that many points.
bool interpolation_points(int alpha, int points_id, std::vector<Rational>* out);

// Fills *out; returns false on invalid (m, k, points_id).
bool generate_winograd(int m, int k, int points_id, WinogradMatrices* out);

}  // namespace mnnb
