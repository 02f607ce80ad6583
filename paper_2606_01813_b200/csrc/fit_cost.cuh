// Offline cost fitting (Section "Offline Cost Profiling", Eq. 12): for every profiled context length, the
// least-squares fit to the measured verification latencies y_0..y_{N-1} (N equally spaced node counts) among all
// convex, non-decreasing sequences.  The paper hands this quadratic program to a generic interior-point solver; here
// it is solved exactly by an active-set method on the GPU, one CTA per context length, everything in fp64.
//
// A sequence is convex and non-decreasing iff f_i = a + sum_k beta_k * max(0, i - k) with beta_k >= 0 (beta_0 the
// first slope, beta_k the slope increase at point k) and a free: a non-negative least-squares problem.  The
// Lawson-Hanson iteration keeps a passive set P of hinges that may be non-zero:
//   outer step   dual w_k = sum_i max(0, i - k) r_i for the residual r = y - f (two suffix scans); stop when no
//                hinge outside P has w_k > 0, else add the one with the largest w_k;
//   inner step   unconstrained least squares on P; if some beta of P would turn negative, move only as far as
//                feasibility allows, drop the hinges that reached zero, and solve again.
// The least-squares problem on P is a continuous piecewise-linear regression with kinks at P (and a flat start if
// hinge 0 is not in P).  It is solved in the basis of hat functions over the kinks, whose normal equations are
// tridiagonal and well conditioned (the hinge basis itself has a condition number ~N^4); their entries come from
// closed forms and from prefix sums of y and i*y, so one solve costs O(|P|).
#pragma once
#include "common.cuh"

namespace cadd {

constexpr int kFitThreads = 256;
constexpr int kFitMaxN = 2048;
constexpr int kFitMaxKnots = kFitMaxN;     // every point may be a kink (data that is convex already)

constexpr int kFitStatusIterCap = 1;       // status bits of the fit
constexpr int kFitStatusKnotCap = 2;

struct FitParams {
    int n_tables, N;
    const double* y;        // [n_tables, N]
    double* fit;            // [n_tables, N]
    int32_t* n_breaks;      // [n_tables] hinges with beta > 0 in the solution (may be NULL)
    int32_t* status;        // [n_tables] (may be NULL)
};

struct FitShared {
    double y[kFitMaxN];
    double r[kFitMaxN];         // residual, then scan scratch
    double beta[kFitMaxN];      // current feasible iterate (dense over hinges)
    double y0[kFitMaxN + 1];    // prefix sums of y
    double y1[kFitMaxN + 1];    // prefix sums of i * y
    unsigned char in_p[kFitMaxN];
    unsigned char banned[kFitMaxN];
    int knots[kFitMaxKnots + 2];            // sorted hinges of P
    double v[kFitMaxKnots + 2];             // node values of the least-squares solution
    double zb[kFitMaxKnots + 2];            // its beta per knot
    double td[kFitMaxKnots + 2], tu[kFitMaxKnots + 2], tc[kFitMaxKnots + 2];   // tridiagonal system
    double part[kFitThreads];
    int parti[kFitThreads];
    double a;                               // current intercept
    double za;                              // intercept of the least-squares solution
    int p;                                  // |P|
    int pick;
    int flag;
};
inline size_t fit_smem_bytes() { return sizeof(FitShared) + 16; }

// In-place inclusive scan of arr[0..n) over the CTA (forward, or backward when reverse): each thread scans a
// contiguous run, the run totals are scanned by thread 0 (256 values), then added back.
__device__ __forceinline__ void fit_scan(FitShared& sh, double* arr, int n, bool reverse) {
    const int tid = threadIdx.x;
    const int per = (n + kFitThreads - 1) / kFitThreads;
    const int lo = tid * per, hi = min(n, lo + per);
    double run = 0.0;
    if (!reverse) { for (int i = lo; i < hi; ++i) { run += arr[i]; arr[i] = run; } }
    else { for (int i = n - 1 - lo; i > n - 1 - hi; --i) { run += arr[i]; arr[i] = run; } }
    sh.part[tid] = run;
    __syncthreads();
    if (tid == 0) {
        double acc = 0.0;
        for (int t = 0; t < kFitThreads; ++t) { const double x = sh.part[t]; sh.part[t] = acc; acc += x; }
    }
    __syncthreads();
    const double add = sh.part[tid];
    if (!reverse) { for (int i = lo; i < hi; ++i) arr[i] += add; }
    else { for (int i = n - 1 - lo; i > n - 1 - hi; --i) arr[i] += add; }
    __syncthreads();
}

// Least squares over the hinges listed in sh.knots[0..p) (sorted): fills sh.v (node values), sh.zb (beta per knot)
// and sh.za.  Executed by thread 0.
__device__ void fit_solve_passive(FitShared& sh, int N) {
    const int p = sh.p;
    if (p == 0) { sh.za = sh.y0[N] / N; return; }
    // nodes x_0 = knots[0], ..., x_{p-1} = knots[p-1], x_p = N - 1
    auto X = [&](int m) { return m < p ? sh.knots[m] : N - 1; };
    for (int m = 0; m <= p; ++m) { sh.td[m] = 0.0; sh.tu[m] = 0.0; sh.tc[m] = 0.0; }
    sh.td[0] += (double)X(0);                 // flat start: points 0 .. x_0 - 1 carry the first node's value
    sh.tc[0] += sh.y0[X(0)];
    for (int m = 0; m < p; ++m) {             // segment m: points x_m .. x_{m+1} - 1, u = (i - x_m) / h
        const int x = X(m);
        const double h = (double)(X(m + 1) - x);
        const double st = h * (h - 1.0) * 0.5, st2 = (h - 1.0) * h * (2.0 * h - 1.0) / 6.0;
        const double C = st2 / (h * h), B = st / h - C, A = h - 2.0 * st / h + C;
        const double sy = sh.y0[X(m + 1)] - sh.y0[x], siy = sh.y1[X(m + 1)] - sh.y1[x];
        const double E = (siy - (double)x * sy) / h, D = sy - E;
        sh.td[m] += A; sh.td[m + 1] += C; sh.tu[m] += B;
        sh.tc[m] += D; sh.tc[m + 1] += E;
    }
    sh.td[p] += 1.0;                          // the last point
    sh.tc[p] += sh.y[N - 1];
    // Thomas algorithm (symmetric positive definite, diagonally dominant enough for any knot set)
    for (int m = 1; m <= p; ++m) {
        const double w = sh.tu[m - 1] / sh.td[m - 1];
        sh.td[m] -= w * sh.tu[m - 1];
        sh.tc[m] -= w * sh.tc[m - 1];
    }
    sh.v[p] = sh.tc[p] / sh.td[p];
    for (int m = p - 1; m >= 0; --m) sh.v[m] = (sh.tc[m] - sh.tu[m] * sh.v[m + 1]) / sh.td[m];
    double prev = 0.0;
    for (int m = 0; m < p; ++m) {
        const double s = (sh.v[m + 1] - sh.v[m]) / (double)(X(m + 1) - X(m));
        sh.zb[m] = s - prev;
        prev = s;
    }
    sh.za = sh.v[0];
}

__global__ void __launch_bounds__(kFitThreads) fit_cost_kernel(FitParams p) {
    extern __shared__ __align__(16) unsigned char fit_smem_raw[];
    FitShared& sh = *reinterpret_cast<FitShared*>(fit_smem_raw);
    const int tid = threadIdx.x, N = p.N, t = blockIdx.x;
    const double* y = p.y + (size_t)t * N;
    double ymax = 0.0;
    for (int i = tid; i < N; i += kFitThreads) {
        const double x = y[i];
        sh.y[i] = x; sh.beta[i] = 0.0; sh.in_p[i] = 0; sh.banned[i] = 0;
        ymax = fmax(ymax, fabs(x));
    }
    sh.part[tid] = ymax;
    __syncthreads();
    if (tid == 0) {
        double m = 0.0;
        for (int q = 0; q < kFitThreads; ++q) m = fmax(m, sh.part[q]);
        sh.part[0] = m;
        sh.p = 0; sh.flag = 0;
    }
    __syncthreads();
    const double scale = fmax(sh.part[0], 1e-300);
    __syncthreads();
    // prefix sums of y and i*y (exclusive, N + 1 entries)
    for (int i = tid; i < N; i += kFitThreads) { sh.y0[i + 1] = sh.y[i]; sh.y1[i + 1] = (double)i * sh.y[i]; }
    if (tid == 0) { sh.y0[0] = 0.0; sh.y1[0] = 0.0; }
    __syncthreads();
    fit_scan(sh, sh.y0 + 1, N, false);
    fit_scan(sh, sh.y1 + 1, N, false);
    if (tid == 0) sh.a = sh.y0[N] / N;       // P empty: the constant fit
    __syncthreads();

    const double tol = 1e-13 * scale * (double)N * (double)N;      // on w_k = sum_i max(0, i-k) r_i
    int status = 0;
    const int max_outer = 4 * N + 16;
    for (int outer = 0; outer < max_outer && N > 1; ++outer) {
        // ---- residual of the current iterate (a, beta): f_i = a + sum_k beta_k max(0, i - k) ----
        // slopes = prefix sum of beta, f = a + exclusive prefix sum of slopes; both through the scan helper on r
        for (int i = tid; i < N; i += kFitThreads) sh.r[i] = i < N - 1 ? sh.beta[i] : 0.0;
        __syncthreads();
        fit_scan(sh, sh.r, N, false);                               // r[i] = slope of segment i -> i+1
        fit_scan(sh, sh.r, N, false);                               // r[i] = f_{i+1} - a
        {
            const int per = (N + kFitThreads - 1) / kFitThreads;    // shift by one: f_i = a + r[i-1]
            double carry[ (kFitMaxN + kFitThreads - 1) / kFitThreads ];
            const int lo = tid * per, hi = min(N, lo + per);
            for (int i = lo; i < hi; ++i) carry[i - lo] = i > 0 ? sh.r[i - 1] : 0.0;
            __syncthreads();
            for (int i = lo; i < hi; ++i) sh.r[i] = sh.y[i] - (sh.a + carry[i - lo]);
            __syncthreads();
        }
        // ---- dual: w_k = sum_{i>k} (i - k) r_i = sum_{m>=k} S1[m], S1[m] = sum_{i>m} r_i ----
        fit_scan(sh, sh.r, N, true);                                // r[i] = sum_{j>=i} r_j
        {
            const int per = (N + kFitThreads - 1) / kFitThreads;
            double carry[ (kFitMaxN + kFitThreads - 1) / kFitThreads ];
            const int lo = tid * per, hi = min(N, lo + per);
            for (int i = lo; i < hi; ++i) carry[i - lo] = i + 1 < N ? sh.r[i + 1] : 0.0;   // S1[i] = sum_{j>i} r_j
            __syncthreads();
            for (int i = lo; i < hi; ++i) sh.r[i] = carry[i - lo];
            __syncthreads();
        }
        fit_scan(sh, sh.r, N, true);                                // r[k] = w_k  (k = 0..N-2; r[N-1] = 0)
        // ---- the hinge outside P with the largest dual ----
        double best = tol;
        int best_k = -1;
        for (int k = tid; k < N - 1; k += kFitThreads)
            if (!sh.in_p[k] && !sh.banned[k] && sh.r[k] > best) { best = sh.r[k]; best_k = k; }
        sh.part[tid] = best; sh.parti[tid] = best_k;
        __syncthreads();
        if (tid == 0) {
            double b = tol; int bk = -1;
            for (int q = 0; q < kFitThreads; ++q)
                if (sh.parti[q] >= 0 && (sh.part[q] > b || (sh.part[q] == b && bk >= 0 && sh.parti[q] < bk))) { b = sh.part[q]; bk = sh.parti[q]; }
            sh.pick = bk;
        }
        __syncthreads();
        const int pick = sh.pick;
        if (pick < 0) break;                                        // optimal
        if (sh.p >= kFitMaxKnots) { status |= kFitStatusKnotCap; break; }
        if (outer == max_outer - 1) status |= kFitStatusIterCap;
        // ---- inner loop (thread 0; |P| is small) ----
        if (tid == 0) {
            sh.in_p[pick] = 1;
            bool first = true;
            for (int inner = 0; inner < 2 * kFitMaxKnots; ++inner) {
                int pp = 0;
                for (int k = 0; k < N - 1 && pp < kFitMaxKnots + 1; ++k) if (sh.in_p[k]) sh.knots[pp++] = k;
                sh.p = pp;
                fit_solve_passive(sh, N);
                if (first) {
                    // the hinge just added must come out positive; if rounding says otherwise, leave it out for now
                    int at = 0;
                    while (at < pp && sh.knots[at] != pick) ++at;
                    if (at < pp && !(sh.zb[at] > 0.0)) {
                        sh.in_p[pick] = 0; sh.banned[pick] = 1;
                        int q2 = 0;
                        for (int k = 0; k < N - 1; ++k) if (sh.in_p[k]) sh.knots[q2++] = k;
                        sh.p = q2;
                        sh.flag = 1;                                // no progress from this pick
                        break;
                    }
                    first = false;
                }
                double alpha = 2.0;
                for (int m = 0; m < pp; ++m)
                    if (!(sh.zb[m] > 0.0)) {
                        const double bk = sh.beta[sh.knots[m]];
                        alpha = fmin(alpha, bk / (bk - sh.zb[m]));
                    }
                if (alpha > 1.0) {                                  // the solution on P is feasible: take it
                    for (int m = 0; m < pp; ++m) sh.beta[sh.knots[m]] = sh.zb[m];
                    sh.a = sh.za;
                    sh.flag = 0;
                    break;
                }
                alpha = fmax(alpha, 0.0);
                for (int m = 0; m < pp; ++m) {                      // move as far as feasibility allows
                    const int k = sh.knots[m];
                    double nb = sh.beta[k] + alpha * (sh.zb[m] - sh.beta[k]);
                    if (!(sh.zb[m] > 0.0) && !(nb > 1e-15 * scale)) nb = 0.0;
                    if (nb <= 0.0) { nb = 0.0; sh.in_p[k] = 0; }
                    sh.beta[k] = nb;
                }
                sh.a += alpha * (sh.za - sh.a);
            }
            if (sh.flag == 0)
                for (int k = 0; k < N - 1; ++k) sh.banned[k] = 0;   // progress: earlier refusals may be tried again
        }
        __syncthreads();
    }

    // ---- write the fit of the final iterate ----
    for (int i = tid; i < N; i += kFitThreads) sh.r[i] = i < N - 1 ? sh.beta[i] : 0.0;
    __syncthreads();
    fit_scan(sh, sh.r, N, false);
    fit_scan(sh, sh.r, N, false);
    for (int i = tid; i < N; i += kFitThreads) p.fit[(size_t)t * N + i] = sh.a + (i > 0 ? sh.r[i - 1] : 0.0);
    if (tid == 0) {
        int nb = 0;
        for (int k = 0; k < N - 1; ++k) nb += sh.beta[k] > 0.0;
        if (p.n_breaks) p.n_breaks[t] = nb;
        if (p.status) p.status[t] = status;
    }
}

}  // namespace cadd
