// Pack modelling (Sec. 4.5): Eq. 6, a non-negative least-squares fit of every pack's feature vector by the
// micro-benchmarks' metric vectors, and Eq. 7, the pack's tables as the weighted sums of the micro-benchmarks'
// tables.  Included only by emo_lib.cu.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

constexpr int kModelMaxM = 16;       // micro-benchmarks (the paper uses 12)

struct ModelParams {
    int n_packs, n, m, L;
    const double *B;        // [n][m] metric matrix
    const double *feat;     // [n_packs][n]
    const double *Tb, *Eb;  // [m][L]
    double *x;              // [n_packs][m]
    double *T_out, *E_out;  // [n_packs][L]
    int32_t *status;
};

// One thread per pack.  The problem is tiny (m <= 16 unknowns) and every pack is independent; the Gram matrix
// G = B^T B is the same for all packs and is built once per block in shared memory, so a pack costs B^T b, the
// active-set iterations on (G, c) and the two weighted sums.
//
// Active-set method of Lawson and Hanson on the normal equations: start from x = 0 with every variable held at
// zero; move the variable with the largest positive gradient component w = c - G x into the free set; solve
// the free set's equations G_PP z = c_P (Cholesky); while z has non-positive entries step from x towards z as
// far as feasibility allows and return the variables that reach zero to the held set; accept z; repeat until no
// gradient component is positive.  Every accepted x lowers the objective, so the loop ends; it is also bounded
// by 3 m outer and 3 m inner rounds (status -9 otherwise: never seen).
__global__ void __launch_bounds__(128) emo_pack_model_kernel(ModelParams p)
{
    extern __shared__ double emo_model_smem[];
    const int m = p.m, n = p.n, L = p.L;
    double *G = emo_model_smem;                    // [m][m]
    double *Bs = G + m * m;                        // [n][m]
    double *Ts = Bs + n * m;                       // [m][L]
    double *Es = Ts + m * L;                       // [m][L]
    for (int i = threadIdx.x; i < n * m; i += blockDim.x) Bs[i] = p.B[i];
    for (int i = threadIdx.x; i < m * L; i += blockDim.x) {
        Ts[i] = p.Tb[i];
        Es[i] = p.Eb[i];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < m * m; i += blockDim.x) {
        const int a = i / m, b = i - a * m;
        double s = 0.0;
        for (int r = 0; r < n; ++r) s += Bs[r * m + a] * Bs[r * m + b];
        G[i] = s;
    }
    __syncthreads();
    const int pk = blockIdx.x * blockDim.x + threadIdx.x;
    if (pk >= p.n_packs) return;

    double c[kModelMaxM], x[kModelMaxM], z[kModelMaxM], Lc[kModelMaxM * kModelMaxM];
    int idx[kModelMaxM];
    unsigned free_set = 0;
    double cmax = 0.0;
    for (int i = 0; i < m; ++i) {
        double s = 0.0;
        for (int r = 0; r < n; ++r) s += Bs[r * m + i] * p.feat[(size_t)pk * n + r];
        c[i] = s;
        x[i] = 0.0;
        cmax = fmax(cmax, fabs(s));
    }
    const double tol = 1e-13 * (cmax > 0.0 ? cmax : 1.0);
    bool failed = false;
    for (int outer = 0; outer < 3 * m; ++outer) {
        // the held variable with the largest gradient component
        int j = -1;
        double wj = tol;
        for (int i = 0; i < m; ++i) {
            if (free_set & (1u << i)) continue;
            double w = c[i];
            for (int k = 0; k < m; ++k) w -= G[i * m + k] * x[k];
            if (w > wj) {
                wj = w;
                j = i;
            }
        }
        if (j < 0) break;
        free_set |= 1u << j;
        bool accepted = false;
        for (int inner = 0; inner < 3 * m && !accepted; ++inner) {
            int k = 0;
            for (int i = 0; i < m; ++i)
                if (free_set & (1u << i)) idx[k++] = i;
            // Cholesky of G_PP, then the two triangular solves
            bool ok = true;
            for (int a = 0; a < k && ok; ++a)
                for (int b = 0; b <= a; ++b) {
                    double s = G[idx[a] * m + idx[b]];
                    for (int q = 0; q < b; ++q) s -= Lc[a * kModelMaxM + q] * Lc[b * kModelMaxM + q];
                    if (a == b) {
                        if (s <= 1e-14 * G[idx[a] * m + idx[a]]) { ok = false; break; }
                        Lc[a * kModelMaxM + a] = sqrt(s);
                    } else {
                        Lc[a * kModelMaxM + b] = s / Lc[b * kModelMaxM + b];
                    }
                }
            if (!ok) {
                // the new column depends on the free ones: it cannot improve the fit, hold it again
                free_set &= ~(1u << j);
                accepted = true;
                break;
            }
            for (int a = 0; a < k; ++a) {
                double s = c[idx[a]];
                for (int q = 0; q < a; ++q) s -= Lc[a * kModelMaxM + q] * z[q];
                z[a] = s / Lc[a * kModelMaxM + a];
            }
            for (int a = k - 1; a >= 0; --a) {
                double s = z[a];
                for (int q = a + 1; q < k; ++q) s -= Lc[q * kModelMaxM + a] * z[q];
                z[a] = s / Lc[a * kModelMaxM + a];
            }
            // feasible?  otherwise the longest step towards z that keeps x >= 0
            double alpha = 2.0;
            for (int a = 0; a < k; ++a)
                if (z[a] <= 0.0) {
                    const double xa = x[idx[a]];
                    alpha = fmin(alpha, xa / (xa - z[a]));
                }
            if (alpha > 1.0) {
                for (int a = 0; a < k; ++a) x[idx[a]] = z[a];
                accepted = true;
            } else {
                for (int a = 0; a < k; ++a) {
                    const int i = idx[a];
                    x[i] += alpha * (z[a] - x[i]);
                    if (x[i] <= 0.0 || (z[a] <= 0.0 && x[i] <= 1e-300)) {
                        x[i] = 0.0;
                        free_set &= ~(1u << i);
                    }
                }
                // the variable that set alpha is exactly at zero up to rounding: make sure it leaves
                for (int a = 0; a < k; ++a) {
                    const int i = idx[a];
                    if ((free_set & (1u << i)) && z[a] <= 0.0 && x[i] <= 1e-15 * fabs(z[a])) {
                        x[i] = 0.0;
                        free_set &= ~(1u << i);
                    }
                }
            }
        }
        if (!accepted) { failed = true; break; }
    }
    if (failed && p.status) atomicMin(p.status, -9);
    for (int i = 0; i < m; ++i) p.x[(size_t)pk * m + i] = x[i];
    // Eq. 7
    for (int l = 0; l < L; ++l) {
        double t = 0.0, e = 0.0;
        for (int i = 0; i < m; ++i) {
            t += x[i] * Ts[i * L + l];
            e += x[i] * Es[i * L + l];
        }
        p.T_out[(size_t)pk * L + l] = t;
        p.E_out[(size_t)pk * L + l] = e;
    }
}
