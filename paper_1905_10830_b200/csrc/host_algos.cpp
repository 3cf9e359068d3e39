// Host-side algorithms of the codec library: Huffman code lengths (Section 3.1, "Variable
// length coding"), canonical code assignment, and the symmetric eigensolver used by the fit
// (Section 3: T diagonalises the covariance).  No device code here.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <vector>

#include "tc.h"

int tc_huffman_lengths_host(const uint64_t *counts, int nsym, int lmax, uint8_t *len);
void tc_canonical_codes_host(const uint8_t *len, int nsym, uint32_t *code);
int tc_eigh_host(double *a, int n, double *evals, double *evecs);

namespace {

// Symbols ordered by (weight, symbol).
std::vector<int> sorted_symbols(const std::vector<uint64_t> &w)
{
    std::vector<int> order(w.size());
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return w[a] < w[b]; });
    return order;
}

// Huffman by two FIFO queues: sorted leaves and internal nodes in creation order (their
// weights are non-decreasing).  A leaf wins a tie against an internal node.
void plain_huffman(const std::vector<uint64_t> &w, std::vector<int> &depth)
{
    const int n = (int)w.size();
    const std::vector<int> order = sorted_symbols(w);
    struct Node { uint64_t w; int up; };
    std::vector<Node> node;
    node.reserve(2 * n);
    for (int i = 0; i < n; ++i) node.push_back({w[order[i]], -1});
    size_t leaf_head = 0, inner_head = (size_t)n;
    auto pop_min = [&]() -> int {
        const bool leaf_ok = leaf_head < (size_t)n;
        const bool inner_ok = inner_head < node.size();
        if (leaf_ok && (!inner_ok || node[leaf_head].w <= node[inner_head].w)) return (int)leaf_head++;
        return (int)inner_head++;
    };
    for (int merges = 0; merges < n - 1; ++merges) {
        const int a = pop_min();
        const int b = pop_min();
        const int id = (int)node.size();
        node.push_back({node[a].w + node[b].w, -1});
        node[a].up = id;
        node[b].up = id;
    }
    depth.assign(n, 0);
    for (int i = 0; i < n; ++i) {
        int d = 0;
        for (int v = i; node[v].up >= 0; v = node[v].up) ++d;
        depth[order[i]] = d;
    }
}

// Package-merge: the optimal prefix code with no code longer than lmax.  Each round pairs up
// the current list into packages and merges them with the leaves (a leaf wins a tie); after
// lmax - 1 rounds the 2n - 2 cheapest items are chosen, and a symbol's code length is the
// number of chosen items it is part of.
void limited_huffman(const std::vector<uint64_t> &w, int lmax, std::vector<int> &depth)
{
    const int n = (int)w.size();
    const std::vector<int> order = sorted_symbols(w);
    struct Item { uint64_t w; std::vector<uint16_t> members; };
    std::vector<Item> leaves;
    for (int s : order) leaves.push_back({w[s], {(uint16_t)s}});
    std::vector<Item> cur = leaves;
    for (int round = 1; round < lmax; ++round) {
        std::vector<Item> packages;
        for (size_t i = 0; i + 1 < cur.size(); i += 2) {
            Item p{cur[i].w + cur[i + 1].w, cur[i].members};
            p.members.insert(p.members.end(), cur[i + 1].members.begin(), cur[i + 1].members.end());
            packages.push_back(std::move(p));
        }
        std::vector<Item> merged;
        merged.reserve(leaves.size() + packages.size());
        size_t a = 0, b = 0;
        while (a < leaves.size() || b < packages.size()) {
            if (a < leaves.size() && (b >= packages.size() || leaves[a].w <= packages[b].w))
                merged.push_back(leaves[a++]);
            else
                merged.push_back(std::move(packages[b++]));
        }
        cur.swap(merged);
    }
    depth.assign(n, 0);
    for (int i = 0; i < 2 * n - 2; ++i)
        for (uint16_t s : cur[i].members) depth[s] += 1;
}

}  // namespace

int tc_huffman_lengths_host(const uint64_t *counts, int nsym, int lmax, uint8_t *len)
{
    if (!counts || !len || nsym < 2 || lmax < 1 || lmax > 31 || (1ll << lmax) < nsym) return -1;
    std::vector<uint64_t> w(nsym);
    for (int i = 0; i < nsym; ++i) w[i] = counts[i] + 1;   // every symbol gets a code
    std::vector<int> depth;
    plain_huffman(w, depth);
    if (*std::max_element(depth.begin(), depth.end()) > lmax) limited_huffman(w, lmax, depth);
    for (int i = 0; i < nsym; ++i) len[i] = (uint8_t)depth[i];
    return 0;
}

// Canonical codes: walk the symbols in (length, symbol) order, counting up and shifting left
// whenever the length grows.
void tc_canonical_codes_host(const uint8_t *len, int nsym, uint32_t *code)
{
    std::vector<int> order(nsym);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return len[a] < len[b]; });
    uint32_t next = 0;
    int prev_len = 0;
    bool first = true;
    for (int s : order) {
        if (len[s] == 0) { code[s] = 0; continue; }
        if (!first) next = (next + 1) << (len[s] - prev_len);
        code[s] = next;
        prev_len = len[s];
        first = false;
    }
}

// ---------------------------------------------------------------------------------------
// Symmetric eigensolver: Householder reduction to tridiagonal form, then implicit-shift QR
// sweeps (Wilkinson shift) with deflation; rotations are accumulated into the basis.
// ---------------------------------------------------------------------------------------
int tc_eigh_host(double *a, int n, double *evals, double *evecs)
{
    if (n <= 0) return -1;
    const size_t N = (size_t)n;
    std::vector<double> q(N * N, 0.0);          // accumulates the reflectors, row-major
    for (int i = 0; i < n; ++i) q[i * N + i] = 1.0;
    std::vector<double> v(N), p(N), wv(N);

    for (int k = 0; k + 2 < n; ++k) {
        double norm2 = 0.0;
        for (int i = k + 1; i < n; ++i) norm2 += a[i * N + k] * a[i * N + k];
        const double normx = std::sqrt(norm2);
        if (normx == 0.0) continue;
        const double x0 = a[(k + 1) * N + k];
        const double alpha = (x0 > 0.0) ? -normx : normx;
        for (int i = k + 1; i < n; ++i) v[i] = a[i * N + k];
        v[k + 1] -= alpha;
        double vn2 = 0.0;
        for (int i = k + 1; i < n; ++i) vn2 += v[i] * v[i];
        if (vn2 == 0.0) continue;
        const double inv = 1.0 / std::sqrt(vn2);
        for (int i = k + 1; i < n; ++i) v[i] *= inv;
        // trailing block B <- H B H with H = I - 2 v v^T
        for (int i = k + 1; i < n; ++i) {
            double s = 0.0;
            const double *row = a + i * N;
            for (int j = k + 1; j < n; ++j) s += row[j] * v[j];
            p[i] = s;
        }
        double kc = 0.0;
        for (int i = k + 1; i < n; ++i) kc += v[i] * p[i];
        for (int i = k + 1; i < n; ++i) wv[i] = p[i] - kc * v[i];
        for (int i = k + 1; i < n; ++i) {
            double *row = a + i * N;
            const double vi = 2.0 * v[i], wi = 2.0 * wv[i];
            for (int j = k + 1; j < n; ++j) row[j] -= vi * wv[j] + wi * v[j];
        }
        // column / row k: H x = alpha e1
        a[(k + 1) * N + k] = a[k * N + (k + 1)] = alpha;
        for (int i = k + 2; i < n; ++i) a[i * N + k] = a[k * N + i] = 0.0;
        // Q <- Q H
        for (int i = 0; i < n; ++i) {
            double *row = q.data() + i * N;
            double t = 0.0;
            for (int j = k + 1; j < n; ++j) t += row[j] * v[j];
            t *= 2.0;
            for (int j = k + 1; j < n; ++j) row[j] -= t * v[j];
        }
    }

    std::vector<double> d(N), e(N, 0.0);
    for (int i = 0; i < n; ++i) d[i] = a[i * N + i];
    for (int i = 0; i + 1 < n; ++i) e[i] = a[(i + 1) * N + i];

    // rows of qt = columns of q, so that rotations touch contiguous memory
    std::vector<double> qt(N * N);
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) qt[j * N + i] = q[i * N + j];

    const double eps = 2.220446049250313e-16;
    long long budget = 60ll * n + 200;
    while (true) {
        for (int i = 0; i + 1 < n; ++i)
            if (std::fabs(e[i]) <= eps * (std::fabs(d[i]) + std::fabs(d[i + 1]))) e[i] = 0.0;
        int hi = n - 1;
        while (hi > 0 && e[hi - 1] == 0.0) --hi;
        if (hi == 0) break;
        int lo = hi - 1;
        while (lo > 0 && e[lo - 1] != 0.0) --lo;
        if (--budget < 0) return -2;
        const double dd = 0.5 * (d[hi - 1] - d[hi]);
        const double eh = e[hi - 1];
        const double denom = dd + (dd >= 0.0 ? 1.0 : -1.0) * std::sqrt(dd * dd + eh * eh);
        const double mu = (denom != 0.0) ? d[hi] - eh * eh / denom : d[hi];
        double x = d[lo] - mu, z = e[lo];
        for (int k = lo; k < hi; ++k) {
            const double r = std::hypot(x, z);
            double c = 1.0, s = 0.0;
            if (r != 0.0) { c = x / r; s = -z / r; }
            if (k > lo) e[k - 1] = r;
            const double d1 = d[k], d2 = d[k + 1], ek = e[k];
            d[k] = c * c * d1 - 2.0 * c * s * ek + s * s * d2;
            d[k + 1] = s * s * d1 + 2.0 * c * s * ek + c * c * d2;
            e[k] = c * s * (d1 - d2) + (c * c - s * s) * ek;
            if (k + 1 < hi) {
                z = -s * e[k + 1];
                e[k + 1] = c * e[k + 1];
                x = e[k];
            }
            double *r0 = qt.data() + (size_t)k * N, *r1 = qt.data() + (size_t)(k + 1) * N;
            for (int j = 0; j < n; ++j) {
                const double u0 = r0[j], u1 = r1[j];
                r0[j] = c * u0 - s * u1;
                r1[j] = s * u0 + c * u1;
            }
        }
    }

    std::vector<int> order(n);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int i, int j) { return d[i] > d[j]; });
    for (int j = 0; j < n; ++j) {
        const double *src = qt.data() + (size_t)order[j] * N;
        int big = 0;
        for (int i = 1; i < n; ++i)
            if (std::fabs(src[i]) > std::fabs(src[big])) big = i;
        const double sgn = (src[big] < 0.0) ? -1.0 : 1.0;
        for (int i = 0; i < n; ++i) evecs[(size_t)j * N + i] = sgn * src[i];
        evals[j] = d[order[j]];
    }
    return 0;
}
