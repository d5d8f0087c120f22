// Host-side plan builder: irreps descriptors -> allowed paths -> real Clebsch-Gordan
// coefficients -> sparse records sorted by output coordinate.
//
// Coefficients follow the paper's "Reconstruction of Clebsch Gordan coefficients":
// the top-spin vector |LL> of every irreducible subspace of Y_l (x) Y_l' is obtained
// from the eigenvalue equation J^2 |LL> = L(L+1) |LL>, which is a three-term
// (triangular) recurrence in m, and the remaining |LM> by iterating the lowering
// operator sigma_- (x) 1 + 1 (x) sigma_-.  The complex coefficients are then moved to
// the real harmonic basis and each path is given a canonical sign.
#include "plan.hpp"

#include <algorithm>
#include <cctype>
#include <cmath>
#include <complex>
#include <cstdlib>
#include <cstring>
#include <map>
#include <sstream>

namespace e3j {
namespace {

using ld = long double;
using cld = std::complex<long double>;

inline ld c_plus(int l, int m) { return std::sqrt((ld)(l * (l + 1) - m * (m + 1))); }
inline ld c_minus(int l, int m) { return std::sqrt((ld)(l * (l + 1) - m * (m - 1))); }

// Complex coupling array cg[M+L][m1+l1][m2+l2] = <l1 m1 l2 m2 | L M>.
std::vector<ld> complex_cg_ladder(int l1, int l2, int L) {
    const int n1 = 2 * l1 + 1, n2 = 2 * l2 + 1, nL = 2 * L + 1;
    std::vector<ld> cg((size_t)nL * n1 * n2, 0.0L);
    auto at = [&](int M, int m1, int m2) -> ld& {
        return cg[((size_t)(M + L) * n1 + (m1 + l1)) * n2 + (m2 + l2)];
    };
    // --- top state: V_m multiplies |l1 m, l2 L-m>
    const int m_lo = std::max(-l1, L - l2), m_hi = l1;
    std::vector<ld> V(m_hi - m_lo + 1, 0.0L);
    V[0] = 1.0L;
    for (int m = m_lo; m < m_hi; ++m) {
        const int mp = L - m;
        ld diag = (ld)(L * (L + 1) - l1 * (l1 + 1) - l2 * (l2 + 1) - 2 * m * mp);
        ld num = diag * V[m - m_lo];
        if (m > m_lo) num -= c_plus(l1, m - 1) * c_minus(l2, mp + 1) * V[m - 1 - m_lo];
        V[m + 1 - m_lo] = num / (c_minus(l1, m + 1) * c_plus(l2, mp - 1));
    }
    ld nrm = 0;
    for (ld v : V) nrm += v * v;
    nrm = std::sqrt(nrm);
    // Condon-Shortley: the component with m1 = l1 is positive
    const ld sgn = (V[m_hi - m_lo] < 0) ? -1.0L : 1.0L;
    for (int m = m_lo; m <= m_hi; ++m) at(L, m, L - m) = sgn * V[m - m_lo] / nrm;
    // --- lower: |L,M-1> = (J- (x) 1 + 1 (x) J-) |L,M> / c_-(L,M)
    for (int M = L; M > -L; --M) {
        const ld inv = 1.0L / c_minus(L, M);
        for (int m1 = -l1; m1 <= l1; ++m1) {
            const int m2 = M - m1;
            if (m2 < -l2 || m2 > l2) continue;
            const ld v = at(M, m1, m2);
            if (v == 0.0L) continue;
            if (m1 - 1 >= -l1) at(M - 1, m1 - 1, m2) += inv * c_minus(l1, m1) * v;
            if (m2 - 1 >= -l2) at(M - 1, m1, m2 - 1) += inv * c_minus(l2, m2) * v;
        }
    }
    return cg;
}

// U[m][m'] : real harmonic m as a combination of the complex ones, both indexed m+l.
std::vector<cld> real_basis(int l) {
    const int n = 2 * l + 1;
    std::vector<cld> U((size_t)n * n, cld(0, 0));
    const ld r = 1.0L / std::sqrt(2.0L);
    U[(size_t)l * n + l] = 1.0L;
    for (int m = 1; m <= l; ++m) {
        const ld s = (m % 2) ? -1.0L : 1.0L;
        U[(size_t)(l + m) * n + (l + m)] = cld(s * r, 0);
        U[(size_t)(l + m) * n + (l - m)] = cld(r, 0);
        U[(size_t)(l - m) * n + (l + m)] = cld(0, -s * r);
        U[(size_t)(l - m) * n + (l - m)] = cld(0, r);
    }
    return U;
}

}  // namespace

std::vector<double> real_cg_ladder(int l1, int l2, int L) {
    const int n1 = 2 * l1 + 1, n2 = 2 * l2 + 1, nL = 2 * L + 1;
    const std::vector<ld> cg = complex_cg_ladder(l1, l2, L);
    const std::vector<cld> U1 = real_basis(l1), U2 = real_basis(l2), UL = real_basis(L);
    std::vector<cld> T((size_t)nL * n1 * n2, cld(0, 0));
    // T[M,a,b] = sum UL[M,M'] cg[M',a',b'] conj(U1[a,a']) conj(U2[b,b'])
    for (int Mp = 0; Mp < nL; ++Mp)
        for (int ap = 0; ap < n1; ++ap)
            for (int bp = 0; bp < n2; ++bp) {
                const ld c = cg[((size_t)Mp * n1 + ap) * n2 + bp];
                if (c == 0.0L) continue;
                for (int M = 0; M < nL; ++M) {
                    const cld u = UL[(size_t)M * nL + Mp];
                    if (u == cld(0, 0)) continue;
                    for (int a = 0; a < n1; ++a) {
                        const cld ua = std::conj(U1[(size_t)a * n1 + ap]);
                        if (ua == cld(0, 0)) continue;
                        for (int b = 0; b < n2; ++b) {
                            const cld ub = std::conj(U2[(size_t)b * n2 + bp]);
                            if (ub == cld(0, 0)) continue;
                            T[((size_t)M * n1 + a) * n2 + b] += u * c * ua * ub;
                        }
                    }
                }
            }
    const bool imag = ((l1 + l2 + L) % 2) != 0;
    std::vector<double> R(T.size());
    for (size_t i = 0; i < T.size(); ++i) {
        ld v = imag ? T[i].imag() : T[i].real();
        if (std::fabs(v) < 1e-15L) v = 0.0L;
        R[i] = (double)v;
    }
    for (size_t i = 0; i < R.size(); ++i)
        if (R[i] != 0.0) {
            if (R[i] < 0.0)
                for (double& v : R) v = (v == 0.0) ? 0.0 : -v;
            break;
        }
    return R;
}

namespace {

struct Irrep {
    int mul, l, p;
};

// "128x0e+128x1o" or "0e+1o" (multiplicity defaults to 1)
bool parse_irreps(const char* text, std::vector<Irrep>& out) {
    out.clear();
    if (!text) return false;
    const char* s = text;
    auto skip = [&]() {
        while (*s == ' ' || *s == '\t') ++s;
    };
    while (true) {
        skip();
        if (!std::isdigit((unsigned char)*s)) return false;
        long v = std::strtol(s, const_cast<char**>(&s), 10);
        skip();
        int mul = 1;
        long l = v;
        if (*s == 'x' || *s == 'X') {
            ++s;
            skip();
            if (!std::isdigit((unsigned char)*s)) return false;
            mul = (int)v;
            l = std::strtol(s, const_cast<char**>(&s), 10);
        }
        if (*s != 'e' && *s != 'o') return false;
        const int p = (*s == 'e') ? 1 : -1;
        ++s;
        if (mul <= 0 || l < 0 || l > 64) return false;
        out.push_back({mul, (int)l, p});
        skip();
        if (*s == '+') {
            ++s;
            continue;
        }
        if (*s == '\0') break;
        return false;
    }
    return !out.empty();
}

}  // namespace

int build_plan(e3j_plan& plan, const char* irreps_in, int sh_lmax, const char* irreps_out,
               int out_lmax, unsigned flags) {
    std::vector<Irrep> ins;
    if (!parse_irreps(irreps_in, ins)) return E3J_ERR_BAD_IRREPS;
    if (sh_lmax < 0) return E3J_ERR_INVALID_ARG;
    for (const Irrep& ir : ins)
        if (ir.mul != ins[0].mul) return E3J_ERR_MUL_NOT_UNIFORM;
    int max_l1 = 0;
    for (const Irrep& ir : ins) max_l1 = std::max(max_l1, ir.l);
    if (max_l1 > 8 || sh_lmax > 8) return E3J_ERR_UNSUPPORTED;

    std::vector<std::pair<int, int>> wanted;  // (L, p) in block order
    if (irreps_out) {
        std::vector<Irrep> outs;
        if (!parse_irreps(irreps_out, outs)) return E3J_ERR_BAD_IRREPS;
        for (const Irrep& ir : outs) wanted.push_back({ir.l, ir.p});
    } else {
        const int lim = (out_lmax < 0) ? max_l1 + sh_lmax : out_lmax;
        for (int L = 0; L <= lim; ++L) {
            const int nat = (L % 2 == 0) ? 1 : -1;
            wanted.push_back({L, nat});
            wanted.push_back({L, -nat});
        }
    }
    auto position = [&](int L, int p) -> int {
        for (size_t i = 0; i < wanted.size(); ++i)
            if (wanted[i].first == L && wanted[i].second == p) return (int)i;
        return -1;
    };

    struct Raw {
        int pos, in_index, l2, l1, p1, L, p, x_off;
    };
    std::vector<Raw> raw;
    int x_off = 0;
    for (size_t idx = 0; idx < ins.size(); ++idx) {
        const int l1 = ins[idx].l, p1 = ins[idx].p;
        for (int l2 = 0; l2 <= sh_lmax; ++l2) {
            const int p = p1 * ((l2 % 2 == 0) ? 1 : -1);
            for (int L = std::abs(l1 - l2); L <= l1 + l2; ++L) {
                const int pos = position(L, p);
                if (pos >= 0) raw.push_back({pos, (int)idx, l2, l1, p1, L, p, x_off});
            }
        }
        x_off += 2 * l1 + 1;
    }
    if (raw.empty()) return E3J_ERR_UNSUPPORTED;
    std::stable_sort(raw.begin(), raw.end(), [](const Raw& a, const Raw& b) {
        if (a.pos != b.pos) return a.pos < b.pos;
        if (a.in_index != b.in_index) return a.in_index < b.in_index;
        return a.l2 < b.l2;
    });

    plan.nq = ins[0].mul;
    plan.d = x_off;
    plan.dp = (sh_lmax + 1) * (sh_lmax + 1);
    plan.P = (int)raw.size();
    plan.flags = flags;
    plan.paths.clear();
    plan.rec.clear();
    // Output blocks: one per path, or (E3J_PLAN_COLLAPSE_OUTPUTS) one per distinct (L, p), shared by all
    // the paths that land on it.  The paths are sorted by output irrep, so those paths are neighbours.
    const bool collapse = (flags & E3J_PLAN_COLLAPSE_OUTPUTS) != 0;
    int out_off = 0, next_off = 0;
    for (int k = 0; k < plan.P; ++k) {
        const Raw& r = raw[k];
        const bool same_block = collapse && k > 0 && raw[k - 1].L == r.L && raw[k - 1].p == r.p;
        if (!same_block) out_off = next_off;
        e3j_path_info_t pi{r.in_index, r.l1, r.p1, r.l2, r.L, r.p, r.x_off, r.l2 * r.l2, out_off};
        plan.paths.push_back(pi);
        const std::vector<double> T = real_cg_ladder(r.l1, r.l2, r.L);
        const int n1 = 2 * r.l1 + 1, n2 = 2 * r.l2 + 1, nL = 2 * r.L + 1;
        for (int M = 0; M < nL; ++M)
            for (int a = 0; a < n1; ++a)
                for (int b = 0; b < n2; ++b) {
                    const double v = T[((size_t)M * n1 + a) * n2 + b];
                    if (v != 0.0) plan.rec.push_back({out_off + M, r.x_off + a, pi.y_off + b, k, v});
                }
        if (!same_block) next_off = out_off + nL;
    }
    plan.D = next_off;
    if (plan.D > 255 || plan.d > 255 || plan.dp > 255 || plan.P > 255) return E3J_ERR_UNSUPPORTED;
    std::sort(plan.rec.begin(), plan.rec.end(), [](const Record& a, const Record& b) {
        if (a.i0 != b.i0) return a.i0 < b.i0;
        if (a.i3 != b.i3) return a.i3 < b.i3;   // (only collapsed plans have several paths per output row)
        if (a.i1 != b.i1) return a.i1 < b.i1;
        return a.i2 < b.i2;
    });
    plan.n_pairs = 0;
    for (size_t i = 0; i < plan.rec.size(); ++i)
        if (i == 0 || plan.rec[i].i0 != plan.rec[i - 1].i0 || plan.rec[i].i1 != plan.rec[i - 1].i1 ||
            plan.rec[i].i3 != plan.rec[i - 1].i3)
            ++plan.n_pairs;

    // canonical signature: multiplicity, input irreps, harmonic degree, output blocks
    std::ostringstream sig;
    sig << plan.nq << "|";
    for (size_t i = 0; i < ins.size(); ++i) sig << (i ? "+" : "") << ins[i].l << (ins[i].p > 0 ? "e" : "o");
    sig << "|" << sh_lmax << "|";
    for (int k = 0; k < plan.P; ++k) {
        const e3j_path_info_t& p = plan.paths[k];
        sig << (k ? "," : "") << p.in_index << ":" << p.l2 << ":" << p.L;
    }
    if (collapse) sig << "|collapsed";
    plan.signature = sig.str();
    return E3J_OK;
}

}  // namespace e3j
