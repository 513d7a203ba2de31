// Host-side compatibility scalars of the reuse-validity gate and the risk certificate (no GPU work).
// Paper: Section 3.2 (discrepancy vector d = [context, size, shape, colour], gate g_tau = prod 1[d_k <= tau_k])
// and Appendix "Risk-Aware Compatibility Decision" (one-sided Clopper-Pearson bound U_alpha(u, n)).
#include <algorithm>
#include <cmath>
#include <vector>

namespace carnator_host {

// CIEDE2000 colour difference between two CIELAB colours (k_L = k_C = k_H = 1).
inline double delta_e00(const double* lab1, const double* lab2) {
    const double pi = 3.14159265358979323846;
    const double L1 = lab1[0], a1 = lab1[1], b1 = lab1[2], L2 = lab2[0], a2 = lab2[1], b2 = lab2[2];
    const double C1 = std::hypot(a1, b1), C2 = std::hypot(a2, b2);
    const double Cm = 0.5 * (C1 + C2);
    const double Cm7 = std::pow(Cm, 7.0);
    const double G = 0.5 * (1.0 - std::sqrt(Cm7 / (Cm7 + 6103515625.0)));          // 25^7
    const double ap1 = (1.0 + G) * a1, ap2 = (1.0 + G) * a2;
    const double Cp1 = std::hypot(ap1, b1), Cp2 = std::hypot(ap2, b2);
    auto hue = [&](double ap, double b) {
        if (ap == 0.0 && b == 0.0) return 0.0;
        double h = std::atan2(b, ap) * 180.0 / pi;
        return h < 0.0 ? h + 360.0 : h;
    };
    const double hp1 = hue(ap1, b1), hp2 = hue(ap2, b2);
    const double dL = L2 - L1, dC = Cp2 - Cp1;
    double dh = 0.0;
    if (Cp1 * Cp2 != 0.0) {
        dh = hp2 - hp1;
        if (dh > 180.0) dh -= 360.0;
        else if (dh < -180.0) dh += 360.0;
    }
    const double dH = 2.0 * std::sqrt(Cp1 * Cp2) * std::sin(0.5 * dh * pi / 180.0);
    const double Lm = 0.5 * (L1 + L2), Cpm = 0.5 * (Cp1 + Cp2);
    double hm = hp1 + hp2;
    if (Cp1 * Cp2 != 0.0) {
        if (std::fabs(hp1 - hp2) <= 180.0) hm *= 0.5;
        else hm = (hp1 + hp2 < 360.0) ? 0.5 * (hp1 + hp2 + 360.0) : 0.5 * (hp1 + hp2 - 360.0);
    }
    const double Tt = 1.0 - 0.17 * std::cos((hm - 30.0) * pi / 180.0) + 0.24 * std::cos(2.0 * hm * pi / 180.0)
                    + 0.32 * std::cos((3.0 * hm + 6.0) * pi / 180.0) - 0.20 * std::cos((4.0 * hm - 63.0) * pi / 180.0);
    const double dtheta = 30.0 * std::exp(-((hm - 275.0) / 25.0) * ((hm - 275.0) / 25.0));
    const double Cpm7 = std::pow(Cpm, 7.0);
    const double Rc = 2.0 * std::sqrt(Cpm7 / (Cpm7 + 6103515625.0));
    const double Sl = 1.0 + 0.015 * (Lm - 50.0) * (Lm - 50.0) / std::sqrt(20.0 + (Lm - 50.0) * (Lm - 50.0));
    const double Sc = 1.0 + 0.045 * Cpm, Sh = 1.0 + 0.015 * Cpm * Tt;
    const double Rt = -std::sin(2.0 * dtheta * pi / 180.0) * Rc;
    const double tl = dL / Sl, tc = dC / Sc, th = dH / Sh;
    return std::sqrt(tl * tl + tc * tc + th * th + Rt * tc * th);
}

// Crop a binary H x W indicator to its tight support box and resample it to res x res (sample at cell centres).
inline bool bbox_normalize(const uint8_t* m, int H, int W, int res, std::vector<uint8_t>& out) {
    int y0 = H, y1 = -1, x0 = W, x1 = -1;
    for (int y = 0; y < H; ++y)
        for (int x = 0; x < W; ++x)
            if (m[y * W + x]) { y0 = std::min(y0, y); y1 = std::max(y1, y); x0 = std::min(x0, x); x1 = std::max(x1, x); }
    out.assign(size_t(res) * res, 0);
    if (y1 < 0) return false;
    const int bh = y1 - y0 + 1, bw = x1 - x0 + 1;
    for (int r = 0; r < res; ++r)
        for (int c = 0; c < res; ++c) {
            const int yy = y0 + std::min(bh - 1, int(((r + 0.5) * bh) / res));
            const int xx = x0 + std::min(bw - 1, int(((c + 0.5) * bw) / res));
            out[size_t(r) * res + c] = m[yy * W + xx] ? 1 : 0;
        }
    return true;
}

// Smallest p with P[X <= u | n, p] <= alpha, i.e. the one-sided upper Clopper-Pearson limit.
inline double clopper_pearson_upper(int u, int n, double alpha) {
    if (u >= n) return 1.0;
    auto cdf = [&](double p) {               // sum_{k<=u} C(n,k) p^k (1-p)^(n-k), terms built up in logs
        double s = 0.0;
        for (int k = 0; k <= u; ++k) {
            double lg = std::lgamma(n + 1.0) - std::lgamma(k + 1.0) - std::lgamma(n - k + 1.0);
            if (k > 0) lg += k * std::log(p);
            if (n - k > 0) lg += (n - k) * std::log1p(-p);
            s += std::exp(lg);
        }
        return s;
    };
    double lo = 0.0, hi = 1.0;
    for (int it = 0; it < 200; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (mid <= 0.0 || mid >= 1.0) break;
        if (cdf(mid) > alpha) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

}  // namespace carnator_host
