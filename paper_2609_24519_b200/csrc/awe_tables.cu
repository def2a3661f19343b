// Host-side configuration records and decomposition tables (Definition 4.1, Algorithm 1 "table
// lookup per value", Appendix A, Section 5.3).  No device code in this file.
#include <cstdlib>
#include <cstring>
#include <map>
#include <tuple>

#include "awe_internal.h"

namespace awe {
namespace {

// The storable integers: E2M1 magnitudes doubled (Section 3.1), ascending.
const int kS[15] = {-12, -8, -6, -4, -3, -2, -1, 0, 1, 2, 3, 4, 6, 8, 12};

bool in_S(int x) {
    int a = std::abs(x);
    return a <= 4 || a == 6 || a == 8 || a == 12;
}

// 4-bit E2M1 pattern (sign, 2 exponent bits, 1 mantissa bit) of an element of S.
uint8_t e2m1_code_of(int s) {
    static const int mag[8] = {0, 1, 2, 3, 4, 6, 8, 12};
    int a = std::abs(s);
    for (int i = 0; i < 8; ++i)
        if (mag[i] == a) return (uint8_t)(i | ((s < 0) ? 8 : 0));
    return 0;
}

void set_vec(int* dst, std::initializer_list<int> v) {
    int i = 0;
    for (int x : v) dst[i++] = x;
}

Scheme make_awe6(int w1, int w2, std::initializer_list<int> ell) {
    // products (P00, P11, P22, P01, P02, P12): single limbs, then pairwise sums (Section 4.3)
    Scheme s;
    s.p = s.q = 3;
    s.r = 6;
    set_vec(s.w, {1, w1, w2});
    set_vec(s.v, {1, w1, w2});
    const int pl[6][3] = {{1, 0, 0}, {0, 1, 0}, {0, 0, 1}, {1, 1, 0}, {1, 0, 1}, {0, 1, 1}};
    for (int k = 0; k < 6; ++k)
        for (int i = 0; i < 3; ++i) s.alpha[k][i] = s.beta[k][i] = pl[k][i];
    int k = 0;
    for (int x : ell) s.ell[k++] = x;
    return s;
}

Scheme make_base13() {
    Scheme s;
    s.p = s.q = 3;
    s.r = 9;
    set_vec(s.w, {1, 13, 169});
    set_vec(s.v, {1, 13, 169});
    int pw[5] = {1, 13, 169, 2197, 28561};
    for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 3; ++j) {
            int k = i * 3 + j;
            s.alpha[k][i] = 1;
            s.beta[k][j] = 1;
            s.ell[k] = pw[i + j];
        }
    return s;
}

Scheme make_awe4() {
    // A = 3 a0 + 5 a1, B = 5 b0 + 3 b1 + 42 b2; 2AB = 35 P1 - 42 P2 + 210 P3 + 15 P4 (Appendix A)
    Scheme s;
    s.p = 2;
    s.q = 3;
    s.r = 4;
    set_vec(s.w, {3, 5});
    set_vec(s.v, {5, 3, 42});
    const int al[4][2] = {{0, 1}, {1, 0}, {1, 2}, {2, 1}};
    const int be[4][3] = {{1, 0, 0}, {0, 1, -1}, {0, 0, 1}, {1, 2, 0}};
    for (int k = 0; k < 4; ++k) {
        for (int i = 0; i < 2; ++i) s.alpha[k][i] = al[k][i];
        for (int i = 0; i < 3; ++i) s.beta[k][i] = be[k][i];
    }
    set_vec(s.ell, {35, -42, 210, 15});
    s.log2D = 1;
    s.a_lo = -8;
    s.a_hi = 7;
    return s;
}

Scheme make_ternary() {
    // A in {-1,0,1} is a single limb; B = b0 + 13 b1 + 169 b2; AB = P0 + 13 P1 + 169 P2 (Section 6.2)
    Scheme s;
    s.p = 1;
    s.q = 3;
    s.r = 3;
    s.w[0] = 1;
    set_vec(s.v, {1, 13, 169});
    for (int k = 0; k < 3; ++k) {
        s.alpha[k][0] = 1;
        s.beta[k][k] = 1;
    }
    set_vec(s.ell, {1, 13, 169});
    s.a_lo = -1;
    s.a_hi = 1;
    return s;
}

Scheme make_int4x4() {
    // x = a0 + 3 a1 on both sides, planes (a0, a1, a0 - a1):
    //   xy = (1 + 3) a0 b0 + (9 + 3) a1 b1 - 3 (a0 - a1)(b0 - b1)
    Scheme s;
    s.p = s.q = 2;
    s.r = 3;
    set_vec(s.w, {1, 3});
    set_vec(s.v, {1, 3});
    const int pl[3][2] = {{1, 0}, {0, 1}, {1, -1}};
    for (int k = 0; k < 3; ++k)
        for (int i = 0; i < 2; ++i) s.alpha[k][i] = s.beta[k][i] = pl[k][i];
    set_vec(s.ell, {4, 12, -3});
    s.a_lo = s.b_lo = -8;
    s.a_hi = s.b_hi = 7;
    return s;
}

Scheme make_fp8sig() {
    // x = a0 + 4 a1 on both sides, planes (a0, a1, a0 - a1):
    //   xy = (1 + 4) a0 b0 + (16 + 4) a1 b1 - 4 (a0 - a1)(b0 - b1)
    // w1 = 4 is the weight whose tables need the smallest plane values (3) over [-15, 15]
    Scheme s;
    s.p = s.q = 2;
    s.r = 3;
    set_vec(s.w, {1, 4});
    set_vec(s.v, {1, 4});
    const int pl[3][2] = {{1, 0}, {0, 1}, {1, -1}};
    for (int k = 0; k < 3; ++k)
        for (int i = 0; i < 2; ++i) s.alpha[k][i] = s.beta[k][i] = pl[k][i];
    set_vec(s.ell, {5, 20, -4});
    s.a_lo = s.b_lo = -16;
    s.a_hi = s.b_hi = 15;
    return s;
}

Scheme make_bf16sig() {
    // A = 4 a0 + 9 a1 + 61 a2 (same for B), planes a0, a1, a2 and a0 + a1: one Karatsuba-type step on the
    // pair (a0, a1), a0 b1 + a1 b0 = (a0+a1)(b0+b1) - a0 b0 - a1 b1, the other cross terms directly:
    //   AB = (16 - 36) a0b0 + (81 - 36) a1b1 + 3721 a2b2 + 36 (a0+a1)(b0+b1)
    //        + 244 (a0b2 + a2b0) + 549 (a1b2 + a2b1)
    // (4, 9, 61) has the smallest plane values (4) among the weights up to (7, 59, 199) whose tables
    // cover [-255, 255] with these planes (coverage 268).
    Scheme s;
    s.p = s.q = 3;
    s.r = 8;
    set_vec(s.w, {4, 9, 61});
    set_vec(s.v, {4, 9, 61});
    const int al[8][3] = {{1, 0, 0}, {0, 1, 0}, {0, 0, 1}, {1, 1, 0}, {1, 0, 0}, {0, 0, 1}, {0, 1, 0}, {0, 0, 1}};
    const int be[8][3] = {{1, 0, 0}, {0, 1, 0}, {0, 0, 1}, {1, 1, 0}, {0, 0, 1}, {1, 0, 0}, {0, 0, 1}, {0, 1, 0}};
    for (int k = 0; k < 8; ++k)
        for (int i = 0; i < 3; ++i) {
            s.alpha[k][i] = al[k][i];
            s.beta[k][i] = be[k][i];
        }
    set_vec(s.ell, {-20, 45, 3721, 36, 244, 244, 549, 549});
    s.a_lo = s.b_lo = -256;
    s.a_hi = s.b_hi = 255;
    return s;
}

Scheme make_fp16sig() {
    // A = a0 + 9 a1 + 71 a2 + 639 a3 (same for B); with P_ij = a_i b_j and
    // Q_kl = (a_2k + 2 a_2k+1)(b_2l + 2 b_2l+1):
    //   2AB = sum_{k,l} 71^(k+l) (-7 P[2k,2l] + 126 P[2k+1,2l+1] + 9 Q[k,l])        (Appendix A)
    Scheme s;
    s.p = s.q = 4;
    s.r = 12;
    set_vec(s.w, {1, 9, 71, 639});
    set_vec(s.v, {1, 9, 71, 639});
    const int pw[3] = {1, 71, 5041};
    int n = 0;
    for (int k = 0; k < 2; ++k)
        for (int l = 0; l < 2; ++l) {
            const int sc = pw[k + l];
            s.alpha[n][2 * k] = 1;
            s.beta[n][2 * l] = 1;
            s.ell[n++] = -7 * sc;
            s.alpha[n][2 * k + 1] = 1;
            s.beta[n][2 * l + 1] = 1;
            s.ell[n++] = 126 * sc;
            s.alpha[n][2 * k] = 1;
            s.alpha[n][2 * k + 1] = 2;
            s.beta[n][2 * l] = 1;
            s.beta[n][2 * l + 1] = 2;
            s.ell[n++] = 9 * sc;
        }
    s.log2D = 1;
    s.a_lo = s.b_lo = -2048;
    s.a_hi = s.b_hi = 2047;
    return s;
}

Scheme make_mixed_fp8() {
    // x = 13 h + 5 eps on both sides; planes h, h + eps (E4M3) and eps (E2M1):
    //   xy = 104 h h' + 65 (h + eps)(h' + eps') - 40 eps eps'                        (Appendix A)
    Scheme s;
    s.p = s.q = 2;
    s.r = 3;
    set_vec(s.w, {13, 5});
    set_vec(s.v, {13, 5});
    const int pl[3][2] = {{1, 0}, {1, 1}, {0, 1}};
    for (int k = 0; k < 3; ++k)
        for (int i = 0; i < 2; ++i) s.alpha[k][i] = s.beta[k][i] = pl[k][i];
    set_vec(s.ell, {104, 65, -40});
    return s;
}

// 8-bit E4M3 pattern (sign, 4 exponent bits with bias 7, 3 mantissa bits) of an integer |v| <= 15.
uint8_t e4m3_code_of(int v) {
    int a = std::abs(v);
    if (a == 0) return 0;
    int e = 0;
    while ((a >> (e + 1)) != 0) ++e;             // a = 1.mmm x 2^e
    const int mant = ((a << 3) >> e) & 7;        // exact for a <= 15
    return (uint8_t)(((v < 0) ? 0x80 : 0) | ((e + 7) << 3) | mant);
}

constexpr int kFp8Cap = 14;  // largest |value| kept in an E4M3 plane (Appendix A: c_A = c_B = 14)

struct Choice {
    int max_abs, sum_abs;
    int limbs[kMaxLimbs];
    bool valid = false;
};

bool better(const Choice& a, const Choice& b, int n) {
    if (!b.valid) return true;
    if (a.max_abs != b.max_abs) return a.max_abs < b.max_abs;
    if (a.sum_abs != b.sum_abs) return a.sum_abs < b.sum_abs;
    for (int i = 0; i < n; ++i)
        if (a.limbs[i] != b.limbs[i]) return a.limbs[i] < b.limbs[i];
    return false;
}

// Enumerate S^n, keep admissible tuples (every stored plane in S), and choose one tuple per
// represented value: smallest largest-|plane|, then smallest sum of |planes|, then the smallest
// limb tuple in lexicographic order.  Values are keyed by (w.a mod m) for residue schemes.
void choose_tuples(int n, const int* weights, int n_planes, const int (*planes)[kMaxLimbs], int modulus,
                   std::map<int, Choice>* out) {
    int idx[kMaxLimbs] = {0};
    for (;;) {
        Choice c;
        int value = 0;
        for (int i = 0; i < n; ++i) {
            c.limbs[i] = kS[idx[i]];
            value += weights[i] * c.limbs[i];
        }
        bool ok = true;
        c.max_abs = 0;
        c.sum_abs = 0;
        for (int j = 0; j < n_planes && ok; ++j) {
            int pv = 0;
            for (int i = 0; i < n; ++i) pv += planes[j][i] * c.limbs[i];
            ok = in_S(pv);
            c.max_abs = std::max(c.max_abs, std::abs(pv));
            c.sum_abs += std::abs(pv);
        }
        if (ok) {
            c.valid = true;
            int key = modulus ? ((value % modulus) + modulus) % modulus : value;
            auto it = out->find(key);
            if (it == out->end() || better(c, it->second, n)) (*out)[key] = c;
        }
        int d = n - 1;
        while (d >= 0 && ++idx[d] == 15) idx[d--] = 0;
        if (d < 0) break;
    }
}

void stored_planes(const Scheme& s, awe_side_t side, SideTable* t) {
    const int n = side == AWE_SIDE_A ? s.p : s.q;
    t->n_planes = 0;
    for (int k = 0; k < s.r; ++k) {
        const int* pl = side == AWE_SIDE_A ? s.alpha[k] : s.beta[k];
        int found = -1;
        for (int j = 0; j < t->n_planes && found < 0; ++j)
            if (!memcmp(t->planes[j], pl, sizeof(int) * n)) found = j;
        if (found < 0) {
            found = t->n_planes++;
            memcpy(t->planes[found], pl, sizeof(int) * n);
        }
        t->index_of_product[k] = found;
    }
}

// Residue schemes (Section 5.3): returns the largest |plane| if a -> a0 + w1 a1 (mod m) is onto.
int two_limb_cover(int m, int w1, int n_planes, const int (*planes)[kMaxLimbs]) {
    int weights[2] = {1, w1};
    std::map<int, Choice> best;
    choose_tuples(2, weights, n_planes, planes, m, &best);
    if ((int)best.size() != m) return -1;
    int c = 0;
    for (auto& kv : best) c = std::max(c, kv.second.max_abs);
    return c;
}

bool make_mod(int m, Scheme* out) {
    if (m < 2 || m > 169) return false;
    Scheme s;
    s.modulus = m;
    // one product: S itself is a complete residue system
    bool seen[256] = {false};
    int count = 0;
    for (int x : kS) {
        int r = ((x % m) + m) % m;
        if (!seen[r]) {
            seen[r] = true;
            ++count;
        }
    }
    if (count == m) {
        s.p = s.q = 1;
        s.r = 1;
        s.w[0] = s.v[0] = 1;
        s.alpha[0][0] = s.beta[0][0] = 1;
        s.ell[0] = 1;
        *out = s;
        return true;
    }
    // three products on two limbs, planes (a0, a1, a0 - a1):
    //   xy = (1 + w1) a0 b0 + (w1^2 + w1) a1 b1 - w1 (a0 - a1)(b0 - b1)
    const int k3[3][kMaxLimbs] = {{1, 0}, {0, 1}, {1, -1}};
    int best_c = 1 << 30, best_w = 0;
    for (int w1 = 1; w1 < m; ++w1) {
        int c = two_limb_cover(m, w1, 3, k3);
        if (c >= 0 && c < best_c) {
            best_c = c;
            best_w = w1;
        }
    }
    if (best_w) {
        s.p = s.q = 2;
        s.r = 3;
        s.w[0] = s.v[0] = 1;
        s.w[1] = s.v[1] = best_w;
        for (int k = 0; k < 3; ++k)
            for (int i = 0; i < 2; ++i) s.alpha[k][i] = s.beta[k][i] = k3[k][i];
        s.ell[0] = (1 + best_w) % m;
        s.ell[1] = (best_w * best_w + best_w) % m;
        s.ell[2] = (m - best_w) % m;
        *out = s;
        return true;
    }
    // three products with a general third plane p a0 + q a1 (|p|, |q| <= 4, p > 0: the sign of a plane
    // is arbitrary), for the moduli no weight covers with a0 - a1.  From
    //   (a0 + w1 a1)(b0 + w1 b1) = a0 b0 + w1 (a0 b1 + a1 b0) + w1^2 a1 b1
    //   (p a0 + q a1)(p b0 + q b1) = p^2 a0 b0 + p q (a0 b1 + a1 b0) + q^2 a1 b1
    // the coefficients are l3 with l3 p q = w1, l1 = 1 - l3 p^2, l2 = w1^2 - l3 q^2 (mod m).  Candidates
    // are ranked by (largest plane value, |p| + |q|, p, q, w1).
    {
        bool in_s[64] = {false};
        for (int x : kS) in_s[x + 32] = true;
        int bp = 0, bq = 0, bw = 0, bl3 = 0, bc = 1 << 30, bsum = 0;
        for (int pp = 1; pp <= 4; ++pp)
            for (int qq = -4; qq <= 4; ++qq) {
                if (qq == 0) continue;
                int admissible = 0;
                for (int a0 : kS)
                    for (int a1 : kS) {
                        const int t = pp * a0 + qq * a1;
                        if (t >= -12 && t <= 12 && in_s[t + 32]) ++admissible;
                    }
                if (admissible < m) continue;  // too few admissible limb pairs to reach every residue
                const int pl[3][kMaxLimbs] = {{1, 0}, {0, 1}, {pp, qq}};
                for (int w1 = 1; w1 < m; ++w1) {
                    int l3 = -1;
                    for (int l = 0; l < m && l3 < 0; ++l)
                        if ((((l * pp * qq - w1) % m) + m) % m == 0) l3 = l;
                    if (l3 < 0) continue;
                    const int c = two_limb_cover(m, w1, 3, pl);
                    if (c < 0) continue;
                    const int sum = pp + std::abs(qq);
                    // lexicographic comparison of (c, |p|+|q|, p, q, w1) with the best so far
                    const int cand[5] = {c, sum, pp, qq, w1}, cur[5] = {bc, bsum, bp, bq, bw};
                    bool better = bw == 0;
                    for (int i = 0; i < 5 && !better; ++i) {
                        if (cand[i] < cur[i]) better = true;
                        else if (cand[i] > cur[i]) break;
                    }
                    if (better) {
                        bc = c; bsum = sum; bp = pp; bq = qq; bw = w1; bl3 = l3;
                    }
                }
            }
        if (bw) {
            s.p = s.q = 2;
            s.r = 3;
            s.w[0] = s.v[0] = 1;
            s.w[1] = s.v[1] = bw;
            const int pl[3][kMaxLimbs] = {{1, 0}, {0, 1}, {bp, bq}};
            for (int k = 0; k < 3; ++k)
                for (int i = 0; i < 2; ++i) s.alpha[k][i] = s.beta[k][i] = pl[k][i];
            auto modm = [m](long long x) { return (int)(((x % m) + m) % m); };
            s.ell[0] = modm(1 - (long long)bl3 * bp * bp);
            s.ell[1] = modm((long long)bw * bw - (long long)bl3 * bq * bq);
            s.ell[2] = modm(bl3);
            *out = s;
            return true;
        }
    }
    // four products on two limbs: all limb pairs, coefficients (1, w1, w1, w1^2)
    const int d2[2][kMaxLimbs] = {{1, 0}, {0, 1}};
    for (int w1 = 1; w1 < m; ++w1) {
        int c = two_limb_cover(m, w1, 2, d2);
        if (c >= 0 && c < best_c) {
            best_c = c;
            best_w = w1;
        }
    }
    if (!best_w) return false;
    s.p = s.q = 2;
    s.r = 4;
    s.w[0] = s.v[0] = 1;
    s.w[1] = s.v[1] = best_w;
    const int ai[4] = {0, 0, 1, 1}, bi[4] = {0, 1, 0, 1};
    for (int k = 0; k < 4; ++k) {
        s.alpha[k][ai[k]] = 1;
        s.beta[k][bi[k]] = 1;
    }
    s.ell[0] = 1;
    s.ell[1] = s.ell[2] = best_w % m;
    s.ell[3] = (best_w * best_w) % m;
    *out = s;
    return true;
}

std::mutex g_mu;
std::map<std::pair<int, int>, Scheme> g_schemes;
std::map<std::tuple<int, int, int, int>, SideTable> g_tables;

}  // namespace

awe_in_dtype_t natural_dtype(int enc, awe_side_t side) {
    if (enc == AWE_ENC_INT4xINT8_AWE4 && side == AWE_SIDE_A) return AWE_I4_IN_I8;
    if (enc == AWE_ENC_INT4xINT4_3) return AWE_I4_IN_I8;
    if (enc == AWE_ENC_FP16SIG_AWE12) return AWE_I16;
    if (enc == AWE_ENC_FP8SIG_3) return AWE_I5_IN_I8;
    if (enc == AWE_ENC_BF16SIG_8) return AWE_I9_IN_I16;
    if (enc == AWE_ENC_TERNARY_INT8_3 && side == AWE_SIDE_A) return AWE_T2_IN_I8;
    return AWE_I8;
}

bool get_scheme(int enc, int modulus, Scheme* out) {
    std::lock_guard<std::mutex> lock(g_mu);
    auto key = std::make_pair(enc, modulus);
    auto it = g_schemes.find(key);
    if (it != g_schemes.end()) {
        *out = it->second;
        return true;
    }
    Scheme s;
    bool ok = false;
    if (enc != AWE_ENC_MOD_M && modulus != 0) return false;
    switch (enc) {
        case AWE_ENC_INT8_AWE6:
        case AWE_ENC_INT8_AWE6_DERIVED:
            s = make_awe6(29, 37, {-65, -261, 259, 29, 37, 1073});
            ok = true;
            break;
        case AWE_ENC_INT8_AWE6_ALT:
            s = make_awe6(11, 39, {-49, -319, 1053, 11, 39, 429});
            ok = true;
            break;
        case AWE_ENC_INT8_BASE13_9:
            s = make_base13();
            ok = true;
            break;
        case AWE_ENC_INT4xINT8_AWE4:
            s = make_awe4();
            ok = true;
            break;
        case AWE_ENC_FP16SIG_AWE12:
            s = make_fp16sig();
            ok = true;
            break;
        case AWE_ENC_INT4xINT4_3:
            s = make_int4x4();
            ok = true;
            break;
        case AWE_ENC_TERNARY_INT8_3:
            s = make_ternary();
            ok = true;
            break;
        case AWE_ENC_INT8_MIXED_FP8_3:
            s = make_mixed_fp8();
            ok = true;
            break;
        case AWE_ENC_FP8SIG_3:
            s = make_fp8sig();
            ok = true;
            break;
        case AWE_ENC_BF16SIG_8:
            s = make_bf16sig();
            ok = true;
            break;
        case AWE_ENC_MOD_M:
            ok = make_mod(modulus, &s);
            break;
        default:
            ok = false;
    }
    if (!ok) return false;
    g_schemes[key] = s;
    *out = s;
    return true;
}

bool get_side_table(int enc, int modulus, awe_side_t side, awe_in_dtype_t dt, const SideTable** out) {
    dt = table_dtype(dt);
    Scheme s;
    if (!get_scheme(enc, modulus, &s)) return false;
    if (enc == AWE_ENC_INT8_AWE6_DERIVED) {
        // The tuples are those of the full record (all six plane values must lie in S); only the limb
        // planes are stored, and a product of two sum planes names the two limb planes it adds.
        const SideTable* full;
        if (!get_side_table(AWE_ENC_INT8_AWE6, modulus, side, dt, &full)) return false;
        std::lock_guard<std::mutex> lock(g_mu);
        auto key = std::make_tuple(enc, modulus, (int)side, (int)dt);
        auto it = g_tables.find(key);
        if (it == g_tables.end()) {
            SideTable t = *full;
            const int n = side == AWE_SIDE_A ? s.p : s.q;
            t.n_planes = n;
            for (int j = 0; j < AWE_MAX_PLANES; ++j)
                for (int i = 0; i < kMaxLimbs; ++i) t.planes[j][i] = (j < n && i == j) ? 1 : 0;
            for (int k = 0; k < s.r; ++k) {
                const int* pl = side == AWE_SIDE_A ? s.alpha[k] : s.beta[k];
                int first = -1, second = -1;
                for (int i = 0; i < n; ++i) {
                    if (pl[i] == 0) continue;
                    if (pl[i] != 1 || second >= 0) return false;  // only sums of two limbs are formed in the kernel
                    (first < 0 ? first : second) = i;
                }
                if (first < 0) return false;
                t.index_of_product[k] = first;
                t.index2_of_product[k] = second;
            }
            for (int b = 0; b < t.entries; ++b) {
                uint64_t word = 0;
                for (int j = 0; j < AWE_MAX_PLANES; ++j) {
                    int8_t& v = t.value[(size_t)b * AWE_MAX_PLANES + j];
                    if (j >= n) {
                        v = 0;
                        continue;
                    }
                    // limb j is the value of the full record's plane with the unit vector e_j
                    int src = -1;
                    for (int q = 0; q < full->n_planes && src < 0; ++q) {
                        bool unit = true;
                        for (int i = 0; i < n; ++i) unit = unit && full->planes[q][i] == (i == j ? 1 : 0);
                        if (unit) src = q;
                    }
                    if (src < 0) return false;
                    v = full->value[(size_t)b * AWE_MAX_PLANES + src];
                    word |= (uint64_t)e2m1_code_of(v) << (8 * j);
                }
                t.lut[b] = word;
            }
            it = g_tables.emplace(key, t).first;
        }
        *out = &it->second;
        return true;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    auto key = std::make_tuple(enc, modulus, (int)side, (int)dt);
    auto it = g_tables.find(key);
    if (it != g_tables.end()) {
        *out = &it->second;
        return true;
    }
    SideTable t;
    t.entries = is_16bit(dt) ? 4096 : 256;
    t.value.assign((size_t)t.entries * AWE_MAX_PLANES, 0);
    t.lut.assign((size_t)t.entries, 0);
    stored_planes(s, side, &t);
    const int n = side == AWE_SIDE_A ? s.p : s.q;
    const int* weights = side == AWE_SIDE_A ? s.w : s.v;
    std::map<int, Choice> best;
    choose_tuples(n, weights, t.n_planes, t.planes, s.modulus, &best);
    const int lo = side == AWE_SIDE_A ? s.a_lo : s.b_lo;
    const int hi = side == AWE_SIDE_A ? s.a_hi : s.b_hi;
    if (enc == AWE_ENC_INT8_MIXED_FP8_3) {
        // Limb h is any integer whose planes h and h + eps fit E4M3 within +-14; eps in S, |eps| <= 8.
        // Same choice rule as choose_tuples: largest |plane|, then sum of |planes|, then (h, eps).
        if (dt != AWE_I8) return false;
        t.bits[0] = t.bits[1] = 8;
        t.c = 0;
        for (int b = 0; b < 256; ++b) {
            const int x = (int)(int8_t)b;
            Choice best_c;
            for (int e : kS) {
                if (std::abs(e) > 8 || (x - 5 * e) % 13 != 0) continue;
                Choice c;
                const int hh = (x - 5 * e) / 13;
                if (std::abs(hh) > kFp8Cap || std::abs(hh + e) > kFp8Cap) continue;
                c.limbs[0] = hh;
                c.limbs[1] = e;
                c.max_abs = std::max(std::max(std::abs(hh), std::abs(hh + e)), std::abs(e));
                c.sum_abs = std::abs(hh) + std::abs(hh + e) + std::abs(e);
                c.valid = true;
                if (better(c, best_c, 2)) best_c = c;
            }
            if (!best_c.valid) return false;
            const int pv[3] = {best_c.limbs[0], best_c.limbs[0] + best_c.limbs[1], best_c.limbs[1]};
            for (int j = 0; j < 3; ++j) {
                t.value[(size_t)b * AWE_MAX_PLANES + j] = (int8_t)pv[j];
                t.c = std::max(t.c, std::abs(pv[j]));
            }
            t.lut[b] = (uint64_t)e4m3_code_of(pv[0]) | ((uint64_t)e4m3_code_of(pv[1]) << 8) |
                       ((uint64_t)e2m1_code_of(pv[2]) << 16);
        }
        auto ins_m = g_tables.emplace(key, t);
        *out = &ins_m.first->second;
        return true;
    }
    t.c = 0;
    for (int b = 0; b < t.entries; ++b) {
        int x = (int)(int8_t)b;
        if (dt == AWE_I4_IN_I8) x = (int)(int8_t)((b & 0xF) << 4) >> 4;  // low nibble, sign-extended
        if (dt == AWE_I5_IN_I8) x = (int)(int8_t)((b & 0x1F) << 3) >> 3; // low 5 bits, sign-extended
        if (dt == AWE_T2_IN_I8 && (x < -1 || x > 1)) x = 0;              // not a ternary value
        if (dt == AWE_I16) x = (int)(int16_t)((b & 0xFFF) << 4) >> 4;     // low 12 bits, sign-extended
        if (dt == AWE_I9_IN_I16) x = (int)(int16_t)((b & 0x1FF) << 7) >> 7;  // low 9 bits, sign-extended
        int key_x = x;
        if (s.modulus) {
            key_x = ((x % s.modulus) + s.modulus) % s.modulus;
        } else if (x < lo || x > hi) {
            return false;  // the record does not cover this dtype's range
        }
        auto f = best.find(key_x);
        if (f == best.end()) return false;
        uint64_t word = 0;
        for (int j = 0; j < t.n_planes; ++j) {
            int pv = 0;
            for (int i = 0; i < n; ++i) pv += t.planes[j][i] * f->second.limbs[i];
            t.value[(size_t)b * AWE_MAX_PLANES + j] = (int8_t)pv;
            t.c = std::max(t.c, std::abs(pv));
            word |= (uint64_t)e2m1_code_of(pv) << (8 * j);
        }
        t.lut[b] = word;
    }
    auto ins = g_tables.emplace(key, t);
    *out = &ins.first->second;
    return true;
}

}  // namespace awe

using namespace awe;

extern "C" awe_status_t awe_encoding_info(int enc, int modulus, awe_encoding_desc* out) {
    if (!out) return AWE_ERR_INVALID_ARG;
    Scheme s;
    if (!get_scheme(enc, modulus, &s)) return AWE_ERR_UNSUPPORTED;
    const SideTable *ta, *tb;
    if (!get_side_table(enc, modulus, AWE_SIDE_A, natural_dtype(enc, AWE_SIDE_A), &ta) ||
        !get_side_table(enc, modulus, AWE_SIDE_B, natural_dtype(enc, AWE_SIDE_B), &tb))
        return AWE_ERR_UNSUPPORTED;
    memset(out, 0, sizeof(*out));
    out->r = s.r;
    out->n_planes_a = ta->n_planes;
    out->n_planes_b = tb->n_planes;
    for (int k = 0; k < s.r; ++k) {
        out->ia[k] = ta->index_of_product[k];
        out->ib[k] = tb->index_of_product[k];
        out->ell[k] = s.ell[k];
        out->ia2[k] = ta->index2_of_product[k];
        out->ib2[k] = tb->index2_of_product[k];
    }
    for (int k = s.r; k < AWE_MAX_PRODUCTS; ++k) out->ia2[k] = out->ib2[k] = -1;
    out->log2D = s.log2D;
    out->modulus = s.modulus;
    out->c_a = ta->c;
    out->c_b = tb->c;
    out->k_star = (int64_t)(1 << 24) / ((int64_t)std::max(1, ta->c) * std::max(1, tb->c));
    out->a_lo = s.a_lo;
    out->a_hi = s.a_hi;
    out->b_lo = s.b_lo;
    out->b_hi = s.b_hi;
    for (int j = 0; j < ta->n_planes; ++j) out->plane_bits_a[j] = ta->bits[j];
    for (int j = 0; j < tb->n_planes; ++j) out->plane_bits_b[j] = tb->bits[j];
    for (int k = 0; k < s.r; ++k) out->fp8[k] = ta->bits[out->ia[k]] == 8;
    return AWE_OK;
}

extern "C" awe_status_t awe_encoding_lut(int enc, int modulus, awe_side_t side, awe_in_dtype_t dt,
                                         int8_t* lut_host) {
    if (!lut_host || (side != AWE_SIDE_A && side != AWE_SIDE_B) || (int)dt < 0 || (int)dt > 6)
        return AWE_ERR_INVALID_ARG;
    const SideTable* t;
    if (!get_side_table(enc, modulus, side, dt, &t)) return AWE_ERR_UNSUPPORTED;
    for (int b = 0; b < t->entries; ++b)
        for (int j = 0; j < t->n_planes; ++j) lut_host[b * t->n_planes + j] = t->value[(size_t)b * AWE_MAX_PLANES + j];
    return AWE_OK;
}

extern "C" size_t awe_planes_bytes(int enc, int modulus, awe_side_t side, int64_t R, int64_t K) {
    if (R <= 0 || K <= 0) return 0;
    const SideTable* t;
    if (!get_side_table(enc, modulus, side, natural_dtype(enc, side), &t)) return 0;
    return (size_t)plane_units(t->bits, t->n_planes) * (size_t)R * (size_t)plane_pitch_bytes(K);
}

extern "C" size_t awe_workspace_bytes(int enc, int modulus, int64_t M, int64_t N, int64_t K) {
    size_t a = awe_planes_bytes(enc, modulus, AWE_SIDE_A, M, K);
    size_t b = awe_planes_bytes(enc, modulus, AWE_SIDE_B, N, K);
    if (!a || !b) return 0;
    return (size_t)round_up((int64_t)a, 256) + (size_t)round_up((int64_t)b, 256);
}

extern "C" const char* awe_status_string(awe_status_t s) {
    switch (s) {
        case AWE_OK: return "ok";
        case AWE_ERR_INVALID_ARG: return "invalid argument";
        case AWE_ERR_UNSUPPORTED: return "unsupported encoding, modulus or dtype";
        case AWE_ERR_WORKSPACE: return "workspace too small";
        case AWE_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
        case AWE_ERR_RANGE: return "result does not fit the output type";
        case AWE_ERR_CUDA: return "CUDA call failed";
        case AWE_ERR_TIMEOUT: return "bounded device wait expired";
    }
    return "unknown status";
}
