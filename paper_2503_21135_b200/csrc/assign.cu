// Offline bit-width assignment (Section IV-A, Algorithm 1): fuzzy c-means over the experts' significance,
// clusters ranked by significance and mapped to precisions, experts in the overlap of two clusters sent to the
// lower precision.  The paper runs this step offline on at most a few hundred experts; it is host code in double
// precision (no device work, no stream), kept in the library so that a caller can go from measured expert loads to
// the bits vector of dynamo_pack_experts or the target vector of dynamo_set_channel_precision through one ABI.
#include <cmath>
#include <cstdint>
#include <vector>

#include "../../include/dynamo.h"

namespace {

// squared Euclidean distance between point i of x and center k of v
inline double dist2(const double* x, const double* v, int dim) {
    double acc = 0.0;
    for (int a = 0; a < dim; ++a) {
        const double t = x[a] - v[a];
        acc += t * t;
    }
    return acc;
}

// Membership update for one point: u_k = 1 / sum_j (d_k / d_j)^(2/(m-1)), written on squared distances as
// u_k = d2_k^(-1/(m-1)) / sum_j d2_j^(-1/(m-1)).  A point on one or more centers shares its membership among them.
void membership_row(const double* xi, const double* v, int c, int dim, double m, double* u) {
    int zeros = 0;
    std::vector<double> d2(c);
    for (int k = 0; k < c; ++k) {
        d2[k] = dist2(xi, v + (size_t)k * dim, dim);
        zeros += d2[k] == 0.0 ? 1 : 0;
    }
    if (zeros) {
        for (int k = 0; k < c; ++k) u[k] = d2[k] == 0.0 ? 1.0 / zeros : 0.0;
        return;
    }
    const double p = -1.0 / (m - 1.0);
    double sum = 0.0;
    for (int k = 0; k < c; ++k) {
        u[k] = std::pow(d2[k], p);
        sum += u[k];
    }
    if (!std::isfinite(sum)) {  // a distance so small that its power overflows: fall back to the ratio form
        for (int k = 0; k < c; ++k) {
            double s = 0.0;
            for (int j = 0; j < c; ++j) s += std::pow(d2[k] / d2[j], -p);
            u[k] = 1.0 / s;
        }
        return;
    }
    for (int k = 0; k < c; ++k) u[k] /= sum;
}

}  // namespace

extern "C" dynamo_status dynamo_assign_bits(const double* x, int32_t n, int32_t dim, int32_t c, double m, double eps,
                                             int32_t max_iter, const double* u0, const double* token_share,
                                             const int32_t* levels, double overlap, int32_t* bits_out,
                                             int32_t* cluster_out, double* v_out, double* u_out, int32_t* iters_out) {
    if (!x || !levels || !bits_out || (!u0 && !token_share)) return DYNAMO_ERR_NULL;
    if (n < 1 || dim < 1 || c < 1 || c > 16 || c > n || max_iter < 1) return DYNAMO_ERR_SHAPE;
    if (!(m > 1.0) || !(eps >= 0.0) || !(overlap >= 0.0)) return DYNAMO_ERR_ARG;
    for (int r = 0; r < c; ++r) {
        const int b = levels[r];
        if (b != 2 && b != 3 && b != 4 && b != 6 && b != 8) return DYNAMO_ERR_BITS;
    }
    for (long long i = 0; i < (long long)n * dim; ++i)
        if (!std::isfinite(x[i])) return DYNAMO_ERR_ARG;

    std::vector<double> U((size_t)n * c), Un((size_t)n * c), V((size_t)c * dim);
    if (u0) {
        for (int i = 0; i < n; ++i) {
            double s = 0.0;
            for (int k = 0; k < c; ++k) {
                const double t = u0[(size_t)i * c + k];
                if (!(t >= 0.0 && t <= 1.0)) return DYNAMO_ERR_ARG;
                s += t;
            }
            if (std::fabs(s - 1.0) > 1e-9) return DYNAMO_ERR_ARG;
        }
        U.assign(u0, u0 + (size_t)n * c);
    } else {
        // memberships of each share against c anchors spread evenly from the smallest to the largest share
        double lo = token_share[0], hi = token_share[0];
        for (int i = 0; i < n; ++i) {
            if (!std::isfinite(token_share[i])) return DYNAMO_ERR_ARG;
            lo = token_share[i] < lo ? token_share[i] : lo;
            hi = token_share[i] > hi ? token_share[i] : hi;
        }
        if (c == 1 || hi == lo) {
            for (auto& t : U) t = 1.0 / c;
        } else {
            std::vector<double> anchors(c);
            for (int k = 0; k < c; ++k) anchors[k] = lo + (hi - lo) * k / (c - 1);
            for (int i = 0; i < n; ++i) membership_row(token_share + i, anchors.data(), c, 1, m, &U[(size_t)i * c]);
        }
    }

    int it = 0;
    for (;;) {
        // centers: v_k = sum_i u_ik^m x_i / sum_i u_ik^m
        for (int k = 0; k < c; ++k) {
            double den = 0.0;
            std::vector<double> num(dim, 0.0);
            for (int i = 0; i < n; ++i) {
                const double w = std::pow(U[(size_t)i * c + k], m);
                den += w;
                for (int a = 0; a < dim; ++a) num[a] += w * x[(size_t)i * dim + a];
            }
            if (!(den > 0.0)) return DYNAMO_ERR_ARG;  // a cluster without any membership has no center
            for (int a = 0; a < dim; ++a) V[(size_t)k * dim + a] = num[a] / den;
        }
        double diff2 = 0.0;
        for (int i = 0; i < n; ++i) {
            membership_row(x + (size_t)i * dim, V.data(), c, dim, m, &Un[(size_t)i * c]);
            for (int k = 0; k < c; ++k) {
                const double t = Un[(size_t)i * c + k] - U[(size_t)i * c + k];
                diff2 += t * t;
            }
        }
        U.swap(Un);
        ++it;
        if (std::sqrt(diff2) < eps || it >= max_iter) break;
    }

    // clusters from the most to the least significant: mean coordinate of the center, then membership mass, then index
    std::vector<int> order(c), rank(c);
    std::vector<double> mean(c, 0.0), mass(c, 0.0);
    for (int k = 0; k < c; ++k) {
        for (int a = 0; a < dim; ++a) mean[k] += V[(size_t)k * dim + a];
        mean[k] /= dim;
        for (int i = 0; i < n; ++i) mass[k] += U[(size_t)i * c + k];
        order[k] = k;
    }
    for (int a = 1; a < c; ++a) {  // insertion sort, stable on the index
        const int k = order[a];
        int b = a - 1;
        while (b >= 0) {
            const int j = order[b];
            const bool k_first = mean[k] > mean[j] || (mean[k] == mean[j] && mass[k] > mass[j]);
            if (!k_first) break;
            order[b + 1] = j;
            --b;
        }
        order[b + 1] = k;
    }
    for (int r = 0; r < c; ++r) rank[order[r]] = r;

    for (int i = 0; i < n; ++i) {
        const double* u = &U[(size_t)i * c];
        // largest and second largest membership; exact ties resolve to the lower precision (higher rank)
        int k1 = -1, k2 = -1;
        for (int k = 0; k < c; ++k) {
            const bool beats1 = k1 < 0 || u[k] > u[k1] || (u[k] == u[k1] && rank[k] > rank[k1]);
            if (beats1) { k2 = k1; k1 = k; continue; }
            const bool beats2 = k2 < 0 || u[k] > u[k2] || (u[k] == u[k2] && rank[k] > rank[k2]);
            if (beats2) k2 = k;
        }
        int chosen = k1;
        if (k2 >= 0 && u[k1] - u[k2] < overlap && rank[k2] > rank[k1]) chosen = k2;  // low precision first
        bits_out[i] = levels[rank[chosen]];
        if (cluster_out) cluster_out[i] = chosen;
    }
    if (v_out) for (size_t i = 0; i < V.size(); ++i) v_out[i] = V[i];
    if (u_out) for (size_t i = 0; i < U.size(); ++i) u_out[i] = U[i];
    if (iters_out) *iters_out = it;
    return DYNAMO_OK;
}
