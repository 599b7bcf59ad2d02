// Calibration path: the "one-time SVD" (Eq. 4, Eq. 5, Eq. 7) through the Gram matrix.
//
//   G = Fstack^T Fstack                accumulated in fp64 over any number of row chunks
//   V_k = top-k eigenvectors of G      block subspace iteration with Rayleigh-Ritz:
//        Z = G Q;  S = Q^T Z;  S = W Theta W^T (parallel cyclic Jacobi);  Q <- Q W;
//        stop when |G v - theta v| <= tol * theta_1 for the k leading pairs;
//        else Q <- orthonormalise(p(G) Q) (Cholesky-QR, applied twice) and repeat, p a Chebyshev
//        polynomial of degree 1 or 2 that damps the spectrum below the block's smallest Ritz value.
//
// Everything runs on the device in fp64 on the plain ALUs; the host only sequences
// launches and reads two numbers per Rayleigh-Ritz step (residual, filter degree).  The eigen-gap at k
// of the power-law spectra met here is ~1e-6 of the leading eigenvalue, so fp32
// anywhere in this path would miss a 1e-4 bound on the principal-angle cosines.
#include <algorithm>
#include <cmath>
#include <mutex>
#include <utility>

#include "internal.cuh"

namespace svdc {

// tensor-core Gram (gram_umma.cu)
bool umma_gram_supported(int64_t M, int D, int64_t ld, int dtype);
int umma_gram_accumulate(const void *F, int64_t M, int D, int64_t ld, double *G, double *scratch, int *status,
                         cudaStream_t s);
size_t umma_gram_scratch_bytes(int D);

namespace {

struct CalibHeader {
    int32_t D, k_max;
    int64_t rows;
    int32_t status;   // SVDCACHE_OK, or the error a kernel of the accumulation recorded
};

// Width of the iterated block: k wanted columns plus guard columns.  (Half as many guard columns
// as wanted ones cut the multiplications by G from 36 to 24 at k = 64 on the power-law spectra met
// here, but the wider Ritz problem cost as much as that saved: 47 -> 46 ms at k = 64, 226 -> 266 ms
// at k = 128.  A quarter it stays.)
int ritz_width(int D, int k) {
    int p = std::max(16, k / 4);
    int m = (k + p + 7) / 8 * 8;
    return std::min(m, D);
}

struct CalibLayout {
    size_t G, gram_scratch, Q, Z, T, S, W, X, theta, resid, scal, dead, partials, partial_bytes, total;
    int m;
};

CalibLayout calib_layout(int D, int k) {
    CalibLayout L;
    L.m = ritz_width(D, k);
    const size_t dm = align_up((size_t)D * L.m * 8, kAlign), mm = align_up((size_t)L.m * L.m * 8, kAlign);
    size_t at = kHeaderBytes;
    L.G = at; at += align_up((size_t)D * D * 8, kAlign);
    L.gram_scratch = at; at += align_up(umma_gram_scratch_bytes(D), kAlign);   // depends on D only, like G
    L.Q = at; at += dm;
    L.Z = at; at += dm;
    L.T = at; at += dm;
    L.S = at; at += mm;
    L.W = at; at += mm;
    L.X = at; at += mm;
    L.theta = at; at += align_up((size_t)L.m * 8, kAlign);
    L.resid = at; at += align_up((size_t)L.m * 8, kAlign);
    L.scal = at; at += kAlign;
    L.dead = at; at += align_up((size_t)L.m * 4, kAlign);
    // partial products of the solver's split GEMMs (see dgemm); small problems do without
    L.partial_bytes = D >= 1024 ? align_up(std::max((size_t)8 * D * L.m, (size_t)96 * L.m * L.m) * 8, kAlign) : 0;
    L.partials = at; at += L.partial_bytes;
    L.total = at;
    return L;
}

int grid_for(int64_t n) { return (int)std::min<int64_t>((n + 255) / 256, 148 * 8); }

template <typename T> __device__ __forceinline__ double to_double(T x);
template <> __device__ __forceinline__ double to_double<double>(double x) { return x; }
template <> __device__ __forceinline__ double to_double<float>(float x) { return (double)x; }
template <> __device__ __forceinline__ double to_double<__nv_bfloat16>(__nv_bfloat16 x) {
    return (double)__bfloat162float(x);
}

// ---------------------------------------------------------------------------------------
// fp64 GEMM on the plain ALUs:  C[i][j] (+)= sum_l A(l, i) * B[l][j],  i < Md, j < Nd, l < L.
//   A_T = true :  A(l, i) = A[l * lda + i]     ("TN": the reduction index is the row of A)
//   A_T = false:  A(l, i) = A[i * lda + l]     ("NN")
// 64 x 64 tile of C per CTA, 4 x 4 outputs per thread, 16-deep shared-memory slabs.
// upper_only: only tiles with tj >= ti are computed (C symmetric, mirrored later).
// The solver's products are tall and skinny (G Q: 48 x 2 tiles; Q^T Z: 2 x 2 tiles, each with
// a reduction 3072 long), far too few CTAs for 148 SMs: with ksplit > 1, blockIdx.y takes a
// slice of the reduction and writes its partial tile to P[y][Md][Nd]; sum_partials_kernel
// adds the slices in order (no atomics: the result does not depend on timing).
// ---------------------------------------------------------------------------------------
constexpr int GT = 64, GK = 16;

template <typename TA, typename TB, bool A_T>
__global__ void __launch_bounds__(256)
dgemm_kernel(const TA *__restrict__ A, int64_t lda, const TB *__restrict__ B, int64_t ldb, double *C,
             int64_t ldc, int Md, int Nd, int64_t L, int accumulate, int upper_only, int ksplit, double *P) {
    __shared__ double As[GK][GT + 2];
    __shared__ double Bs[GK][GT + 2];
    int ti, tj;
    if (upper_only) {
        const int nt = (Md + GT - 1) / GT;
        int rem = blockIdx.x;
        ti = 0;
        while (rem >= nt - ti) { rem -= nt - ti; ++ti; }
        tj = ti + rem;
    } else {
        const int ntj = (Nd + GT - 1) / GT;
        ti = blockIdx.x / ntj;
        tj = blockIdx.x % ntj;
    }
    const int i0 = ti * GT, j0 = tj * GT;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    double acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;

    const int64_t Lc = ksplit > 1 ? ((L + (int64_t)ksplit * GK - 1) / ((int64_t)ksplit * GK)) * GK : L;
    const int64_t l_begin = (int64_t)blockIdx.y * Lc;
    L = l_begin + Lc < L ? l_begin + Lc : L;   // this CTA's slice of the reduction
    for (int64_t l0 = l_begin; l0 < L; l0 += GK) {
        for (int e = threadIdx.x; e < GK * GT; e += 256) {
            int kk, ii;
            if (A_T) { kk = e / GT; ii = e % GT; } else { ii = e / GK; kk = e % GK; }
            const int64_t l = l0 + kk;
            const int i = i0 + ii;
            double v = 0.0;
            if (l < L && i < Md) v = to_double(A_T ? A[l * lda + i] : A[(int64_t)i * lda + l]);
            As[kk][ii] = v;
        }
        for (int e = threadIdx.x; e < GK * GT; e += 256) {
            const int kk = e / GT, jj = e % GT;
            const int64_t l = l0 + kk;
            const int j = j0 + jj;
            Bs[kk][jj] = (l < L && j < Nd) ? to_double(B[l * ldb + j]) : 0.0;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < GK; ++kk) {
            double a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) { a[u] = As[kk][ty * 4 + u]; b[u] = Bs[kk][tx * 4 + u]; }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[u][v] = fma(a[u], b[v], acc[u][v]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int i = i0 + ty * 4 + u;
        if (i >= Md) continue;
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int j = j0 + tx * 4 + v;
            if (j >= Nd) continue;
            if (ksplit > 1) {
                P[((int64_t)blockIdx.y * Md + i) * Nd + j] = acc[u][v];
            } else {
                double *c = C + (int64_t)i * ldc + j;
                *c = accumulate ? (*c + acc[u][v]) : acc[u][v];
            }
        }
    }
}

__global__ void sum_partials_kernel(const double *P, int ksplit, double *C, int64_t ldc, int Md, int Nd, int accumulate) {
    const int64_t n = (int64_t)Md * Nd;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
        double acc = 0.0;
        for (int y = 0; y < ksplit; ++y) acc += P[(int64_t)y * n + e];
        double *c = C + (e / Nd) * ldc + (e % Nd);
        *c = accumulate ? (*c + acc) : acc;
    }
}

// scratch for split reductions (may be empty: then every product is one CTA deep)
struct Partials { double *buf = nullptr; size_t bytes = 0; };

template <typename TA, typename TB, bool A_T>
int dgemm(const TA *A, int64_t lda, const TB *B, int64_t ldb, double *C, int64_t ldc, int Md, int Nd,
          int64_t L, bool accumulate, bool upper_only, cudaStream_t s, Partials ps = Partials()) {
    const int nti = (Md + GT - 1) / GT, ntj = (Nd + GT - 1) / GT;
    const int blocks = upper_only ? nti * (nti + 1) / 2 : nti * ntj;
    // enough CTAs for ~4 per SM, slices at least two slabs deep, and what the scratch holds
    int64_t ks = upper_only ? 1 : (4 * 148 + blocks - 1) / blocks;
    ks = std::min<int64_t>(ks, L / (2 * GK));
    ks = std::min<int64_t>(ks, (int64_t)(ps.bytes / ((size_t)Md * Nd * 8)));
    if (ks < 2 || ps.buf == nullptr) ks = 1;
    dgemm_kernel<TA, TB, A_T><<<dim3(blocks, (unsigned)ks), 256, 0, s>>>(A, lda, B, ldb, C, ldc, Md, Nd, L, accumulate ? 1 : 0,
                                                                        upper_only ? 1 : 0, (int)ks, ps.buf);
    count_launch();
    if (ks > 1) {
        sum_partials_kernel<<<grid_for((int64_t)Md * Nd), 256, 0, s>>>(ps.buf, (int)ks, C, ldc, Md, Nd, accumulate ? 1 : 0);
        count_launch();
    }
    return check_last_launch();
}

__global__ void zero_kernel(double *p, int64_t n) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        p[i] = 0.0;
}

__global__ void init_header_kernel(CalibHeader *h, int D, int k) {
    h->D = D; h->k_max = k; h->rows = 0; h->status = SVDCACHE_OK;
}

// counts the rows of a chunk; a chunk of another width than the accumulation was begun with
// poisons the header, so that the finish refuses it
__global__ void add_rows_kernel(CalibHeader *h, int64_t M, int D) {
    h->rows += M;
    if (h->D != D && h->status == SVDCACHE_OK) h->status = SVDCACHE_ERR_WORKSPACE;
}

// lower <- upper (mode 0), or S <- (S + S^T)/2 (mode 1)
__global__ void symmetrize_kernel(double *A, int n, int mode) {
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < (int64_t)n * n;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int i = (int)(e / n), j = (int)(e % n);
        if (j < i) {
            if (mode == 0) {
                A[(int64_t)i * n + j] = A[(int64_t)j * n + i];
            } else {
                const double v = 0.5 * (A[(int64_t)i * n + j] + A[(int64_t)j * n + i]);
                A[(int64_t)i * n + j] = v;
                A[(int64_t)j * n + i] = v;
            }
        }
    }
}

__global__ void trace_kernel(const double *G, int n, double *out) {
    __shared__ double red[256];
    double s = 0.0;
    for (int i = threadIdx.x; i < n; i += 256) s += G[(int64_t)i * n + i];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = red[0];
}

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// start block: entries uniform in (-1, 1) from a counter hash (deterministic)
__global__ void init_block_kernel(double *Q, int64_t n) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        Q[i] = (double)(mix64((uint64_t)i) >> 11) * (2.0 / 9007199254740992.0) - 1.0;
}

// ---------------------------------------------------------------------------------------
// Cholesky-QR helper on the m x m Gram matrix S = Z^T Z of a block (one CTA):
//   d_j = 1/sqrt(S_jj);  S' = d S d (unit diagonal);  S' = L L^T;  XT = d L^-T,
// so that Z XT has orthonormal columns.  Scaling first makes the factorisation depend on
// the angles between the columns only, not on their norms (which span lambda_1..lambda_m).
// A column that is numerically dependent on the ones before it (scaled pivot <= 1e-10)
// or is zero is marked dead: its output column is zero and the caller re-seeds it.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) chol_inv_kernel(double *S, double *XT, int m, int *dead) {
    __shared__ double s_dinv[384];
    __shared__ int s_dead[384];
    __shared__ double s_d;
    const int tid = threadIdx.x, nt = blockDim.x;
    for (int j = tid; j < m; j += nt) {
        const double p = S[(int64_t)j * m + j];
        const bool ok = (p > 0.0) && isfinite(p);
        s_dinv[j] = ok ? 1.0 / sqrt(p) : 0.0;
        s_dead[j] = ok ? 0 : 1;
    }
    __syncthreads();
    for (int e = tid; e < m * m; e += nt) {
        const int i = e / m, j = e % m;
        S[e] = S[e] * s_dinv[i] * s_dinv[j];
    }
    __syncthreads();
    for (int j = 0; j < m; ++j) {
        if (tid == 0) {
            const double p = S[(int64_t)j * m + j];
            if (s_dead[j] || !(p > 1e-10)) { s_dead[j] = 1; s_d = 0.0; S[(int64_t)j * m + j] = 1.0; }
            else { s_d = sqrt(p); S[(int64_t)j * m + j] = s_d; }
        }
        __syncthreads();
        const double d = s_d;
        if (d == 0.0) {   // dead column: no coupling to the rest
            for (int i = j + 1 + tid; i < m; i += nt) S[(int64_t)i * m + j] = 0.0;
            __syncthreads();
            continue;
        }
        const double inv = 1.0 / d;
        for (int i = j + 1 + tid; i < m; i += nt) S[(int64_t)i * m + j] *= inv;
        __syncthreads();
        // trailing update of the lower triangle: S[i][l] -= L[i][j] L[l][j], j < l <= i
        const int rem = m - j - 1;
        for (int e = tid; e < rem * rem; e += nt) {
            const int i = j + 1 + e / rem, l = j + 1 + e % rem;
            if (l <= i) S[(int64_t)i * m + l] -= S[(int64_t)i * m + j] * S[(int64_t)l * m + j];
        }
        __syncthreads();
    }
    // X = L^-1 by forward substitution, one column c per thread, stored as row c of XT
    for (int c = tid; c < m; c += nt) {
        for (int i = 0; i < c; ++i) XT[(int64_t)c * m + i] = 0.0;
        XT[(int64_t)c * m + c] = 1.0 / S[(int64_t)c * m + c];
        for (int i = c + 1; i < m; ++i) {
            double acc = 0.0;
            for (int l = c; l < i; ++l) acc += S[(int64_t)i * m + l] * XT[(int64_t)c * m + l];
            XT[(int64_t)c * m + i] = -acc / S[(int64_t)i * m + i];
        }
    }
    __syncthreads();
    // XT[l][j] = d_l * X[j][l]; dead output columns are zeroed
    for (int e = tid; e < m * m; e += nt) {
        const int l = e / m, j = e % m;
        XT[e] = s_dead[j] ? 0.0 : XT[e] * s_dinv[l];
    }
    for (int j = tid; j < m; j += nt) dead[j] = s_dead[j];
}
// Indexing: XT[c][i] holds X[i][c] = (L^-1)[i][c], i.e. (L^-T)[c][i]; the product Z XT
// reads B[l][j] = XT[l][j] = d_l (L^-T)[l][j].

// The same result with the matrix in shared memory (m <= 160), for the sizes the solver runs at:
// the global-memory version above spends its time in ~3 m barriers around L2 round trips and in
// a forward substitution that keeps m threads busy.  Here
//   - the factorisation takes one barrier per column: at step j every thread reads the pivot for
//     itself, the trailing block is updated with the still unscaled column j (factor 1 / pivot),
//     and column j is scaled one step later, when nobody reads it any more;
//   - L is inverted in place from the last column backwards: column j of L^-1 is minus the
//     already inverted trailing block times column j of L, a row per warp.
// Rows are padded to an odd stride so that column accesses do not collide in the banks.
constexpr int kCholSmemRitz = 160;
__global__ void __launch_bounds__(1024) chol_inv_smem_kernel(const double *S, double *XT, int m, int *dead) {
    extern __shared__ double chol_dyn[];
    double *A = chol_dyn;
    __shared__ double s_dinv[kCholSmemRitz], s_diag[kCholSmemRitz];
    __shared__ int s_dead0[kCholSmemRitz], s_dead[kCholSmemRitz];
    const int tid = threadIdx.x, nt = blockDim.x, ty = tid >> 5, tx = tid & 31;
    const int ld = m + 1;
    for (int j = tid; j < m; j += nt) {
        const double p = S[(int64_t)j * m + j];
        const bool ok = (p > 0.0) && isfinite(p);
        s_dinv[j] = ok ? 1.0 / sqrt(p) : 0.0;
        s_dead0[j] = ok ? 0 : 1;
    }
    __syncthreads();
    for (int e = tid; e < m * m; e += nt) {
        const int i = e / m, j = e % m;
        A[i * ld + j] = S[e] * s_dinv[i] * s_dinv[j];
    }
    __syncthreads();
    double inv_prev = 0.0;
    for (int j = 0; j < m; ++j) {
        const double p = A[j * ld + j];
        const bool dj = s_dead0[j] || !(p > 1e-10);
        const double d = dj ? 1.0 : sqrt(p);
        const double inv = dj ? 0.0 : 1.0 / d;
        if (tid == 0) { s_dead[j] = dj ? 1 : 0; s_diag[j] = d; }
        if (j > 0)   // column j - 1 becomes L (zero for a dead column: no coupling to the rest)
            for (int i = j + tid; i < m; i += nt) A[i * ld + j - 1] = inv_prev == 0.0 ? 0.0 : A[i * ld + j - 1] * inv_prev;
        if (!dj) {   // trailing update of the lower triangle: A[i][l] -= L[i][j] L[l][j], j < l <= i
            const double inv2 = inv * inv;
            for (int i = j + 1 + ty; i < m; i += 32) {
                const double aij = A[i * ld + j] * inv2;
                for (int l = j + 1 + tx; l <= i; l += 32) A[i * ld + l] -= aij * A[l * ld + j];
            }
        }
        inv_prev = inv;
        __syncthreads();
    }
    // diagonal of L^-1 into the diagonal of A
    for (int j = tid; j < m; j += nt) A[j * ld + j] = 1.0 / s_diag[j];
    __syncthreads();
    for (int j = m - 2; j >= 0; --j) {
        const double xjj = A[j * ld + j];
        double mine[(kCholSmemRitz + 31) / 32];
        int n = 0;
        for (int i = j + 1 + ty; i < m; i += 32, ++n) {   // X[i][j] = -x_jj sum_{j < l <= i} X[i][l] L[l][j]
            double acc = 0.0;
            for (int l = j + 1 + tx; l <= i; l += 32) acc += A[i * ld + l] * A[l * ld + j];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
            mine[n] = -xjj * acc;
        }
        __syncthreads();   // column j of L has been read by everyone
        n = 0;
        for (int i = j + 1 + ty; i < m; i += 32, ++n)
            if (tx == 0) A[i * ld + j] = mine[n];
        __syncthreads();
    }
    // XT[l][j] = d_l X[j][l] for j >= l, zero above; dead output columns are zeroed
    for (int e = tid; e < m * m; e += nt) {
        const int l = e / m, j = e % m;
        XT[e] = (s_dead[j] || j < l) ? 0.0 : A[j * ld + l] * s_dinv[l];
    }
    for (int j = tid; j < m; j += nt) dead[j] = s_dead[j];
}

// fresh pseudo-random entries for the columns marked dead (salted by `salt`)
__global__ void reseed_dead_kernel(double *Q, int D, int m, const int *dead, uint64_t salt) {
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < (int64_t)D * m;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int j = (int)(e % m);
        if (dead[j]) Q[e] = (double)(mix64((uint64_t)e ^ (salt * 0x9E3779B97F4A7C15ull)) >> 11) * (2.0 / 9007199254740992.0) - 1.0;
    }
}

// ---------------------------------------------------------------------------------------
// Eigen-decomposition of the m x m symmetric Rayleigh-Ritz matrix by parallel cyclic
// Jacobi (round-robin ordering: m/2 disjoint plane rotations per round).  One CTA.
//   S   in: symmetric matrix (destroyed)     W   scratch m x m
//   Wout out: eigenvectors as columns, ordered by descending eigenvalue
//   theta out: eigenvalues, descending       sweeps_out: sweeps used
// A round applies J^T S J for J = product of the round's rotations: the 2 x 2 block of S
// that pairs rotation A's rows with rotation B's columns becomes J_A^T S_AB J_B, so all
// (m/2)^2 blocks update independently.  m must be even.
// ---------------------------------------------------------------------------------------
constexpr int kMaxRitz = 384;
constexpr int kJacobiThreads = 1024;
constexpr size_t kJacobiSmemMax = 200 * 1024;   // S and W of the Ritz problem in shared memory when they fit (m <= 113)

__global__ void __launch_bounds__(1024)
jacobi_kernel(double *S_g, double *W_g, double *Wout, double *theta, int m, double *sweeps_out, int in_smem) {
    // A round is a handful of dependent accesses between barriers: with S and W in global memory
    // each costs an L2 round trip (~1.4 ms per call at m = 80); when both fit they live in shared
    // memory for the whole call.
    extern __shared__ double jacobi_dyn[];
    double *S = in_smem ? jacobi_dyn : S_g;
    double *W = in_smem ? jacobi_dyn + (size_t)m * m : W_g;
    if (in_smem) {
        for (int e = threadIdx.x; e < m * m; e += blockDim.x) S[e] = S_g[e];
    }
    __shared__ double cs_c[kMaxRitz / 2], cs_s[kMaxRitz / 2];
    __shared__ int pr_p[kMaxRitz / 2], pr_q[kMaxRitz / 2];
    __shared__ int s_rot;
    __shared__ double s_diag[kMaxRitz];
    __shared__ int s_rank[kMaxRitz];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int h = m / 2;
    for (int e = tid; e < m * m; e += nt) W[e] = (e / m == e % m) ? 1.0 : 0.0;
    __syncthreads();
    int sweep = 0;
    for (; sweep < 40; ++sweep) {
        if (tid == 0) s_rot = 0;
        __syncthreads();
        for (int r = 0; r < m - 1; ++r) {
            if (tid < h) {
                int p, q;
                if (tid == 0) { p = m - 1; q = r; }
                else { p = (r + tid) % (m - 1); q = (r - tid + (m - 1)) % (m - 1); }
                if (p > q) { const int t = p; p = q; q = t; }
                pr_p[tid] = p; pr_q[tid] = q;
                const double app = S[(int64_t)p * m + p], aqq = S[(int64_t)q * m + q], apq = S[(int64_t)p * m + q];
                double c = 1.0, s = 0.0;
                // (thresholds on squares: this chain of fp64 divisions and roots is the serial part of
                // every round, so it does without the square root of |app aqq|)
                const double pq2 = apq * apq, dd = fabs(app * aqq);
                if (apq != 0.0 && pq2 > 1e-34 * dd) {
                    const double tau = (aqq - app) / (2.0 * apq);
                    const double t = (tau >= 0.0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
                    c = rsqrt(1.0 + t * t);
                    s = t * c;
                    if (pq2 > 1e-30 * dd) atomicAdd(&s_rot, 1);
                }
                cs_c[tid] = c; cs_s[tid] = s;
            }
            __syncthreads();
            // S_AB <- J_A^T S_AB J_B with J = [[c, s], [-s, c]] on the (p, q) plane
            for (int e = tid; e < h * h; e += nt) {
                const int A = e / h, B = e % h;
                const int p = pr_p[A], q = pr_q[A], u = pr_p[B], v = pr_q[B];
                const double ca = cs_c[A], sa = cs_s[A], cb = cs_c[B], sb = cs_s[B];
                double spu = S[(int64_t)p * m + u], spv = S[(int64_t)p * m + v];
                double squ = S[(int64_t)q * m + u], sqv = S[(int64_t)q * m + v];
                // rows: (p, q) <- (c p - s q, s p + c q)
                const double rpu = ca * spu - sa * squ, rpv = ca * spv - sa * sqv;
                const double rqu = sa * spu + ca * squ, rqv = sa * spv + ca * sqv;
                // columns: (u, v) <- (c u - s v, s u + c v)
                S[(int64_t)p * m + u] = cb * rpu - sb * rpv;
                S[(int64_t)p * m + v] = sb * rpu + cb * rpv;
                S[(int64_t)q * m + u] = cb * rqu - sb * rqv;
                S[(int64_t)q * m + v] = sb * rqu + cb * rqv;
            }
            // W <- W J (columns)
            for (int e = tid; e < m * h; e += nt) {
                const int i = e / h, B = e % h;
                const int u = pr_p[B], v = pr_q[B];
                const double cb = cs_c[B], sb = cs_s[B];
                const double wu = W[(int64_t)i * m + u], wv = W[(int64_t)i * m + v];
                W[(int64_t)i * m + u] = cb * wu - sb * wv;
                W[(int64_t)i * m + v] = sb * wu + cb * wv;
            }
            __syncthreads();
        }
        if (s_rot == 0) { ++sweep; break; }
        __syncthreads();
    }
    // order by descending eigenvalue (rank sort; ties by index)
    for (int i = tid; i < m; i += nt) s_diag[i] = S[(int64_t)i * m + i];
    __syncthreads();
    for (int j = tid; j < m; j += nt) {
        int rk = 0;
        const double x = s_diag[j];
        for (int i = 0; i < m; ++i) rk += (s_diag[i] > x) || (s_diag[i] == x && i < j);
        s_rank[j] = rk;
        theta[rk] = x;
    }
    __syncthreads();
    for (int e = tid; e < m * m; e += nt) {
        const int i = e / m, j = e % m;
        Wout[(int64_t)i * m + s_rank[j]] = W[e];
    }
    if (tid == 0 && sweeps_out) *sweeps_out = (double)sweep;
}

// ---------------------------------------------------------------------------------------
// The same eigen-decomposition for Ritz matrices whose S and W do not fit in shared memory
// together (113 < m <= 160, i.e. k = 128): S alone lives in shared memory, and the eigenvector
// matrix is not touched during the sweeps at all -- every rotation's (c, s) goes to a log in
// global memory (the pairs of a round follow from its number), and apply_rotations_kernel
// forms W = J_1 J_2 ... afterwards, a warp per row of W, rows being independent.  With both
// matrices in global memory a call took 13.6 ms at m = 160, every round a chain of L2 round trips.
//   head[0] = rounds logged, head[1 + j] = rank of eigenvalue j (descending); log after kJacobiLogHead bytes
// ---------------------------------------------------------------------------------------
constexpr int kJacobiLogRitz = 160;
constexpr size_t kJacobiLogHead = 1024;
constexpr int kJacobiMaxSweeps = 40;

__device__ __forceinline__ void jacobi_pair(int r, int B, int m, int &p, int &q) {
    if (B == 0) { p = m - 1; q = r; }
    else { p = (r + B) % (m - 1); q = (r - B + (m - 1)) % (m - 1); }
    if (p > q) { const int t = p; p = q; q = t; }
}

__global__ void __launch_bounds__(1024)
jacobi_logged_kernel(const double *S_g, double *theta, int m, double *sweeps_out, int *head, double2 *log) {
    extern __shared__ double jacobi_dyn[];
    double *S = jacobi_dyn;
    __shared__ double cs_c[kJacobiLogRitz / 2], cs_s[kJacobiLogRitz / 2];
    __shared__ int pr_p[kJacobiLogRitz / 2], pr_q[kJacobiLogRitz / 2];
    __shared__ int s_rot;
    __shared__ double s_diag[kJacobiLogRitz];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int h = m / 2;
    for (int e = tid; e < m * m; e += nt) S[e] = S_g[e];
    __syncthreads();
    int sweep = 0, round = 0;
    for (; sweep < kJacobiMaxSweeps; ++sweep) {
        if (tid == 0) s_rot = 0;
        __syncthreads();
        for (int r = 0; r < m - 1; ++r, ++round) {
            if (tid < h) {
                int p, q;
                jacobi_pair(r, tid, m, p, q);
                pr_p[tid] = p; pr_q[tid] = q;
                const double app = S[p * m + p], aqq = S[q * m + q], apq = S[p * m + q];
                double c = 1.0, sn = 0.0;
                const double pq2 = apq * apq, dd = fabs(app * aqq);
                if (apq != 0.0 && pq2 > 1e-34 * dd) {
                    const double tau = (aqq - app) / (2.0 * apq);
                    const double t = (tau >= 0.0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
                    c = rsqrt(1.0 + t * t);
                    sn = t * c;
                    if (pq2 > 1e-30 * dd) atomicAdd(&s_rot, 1);
                }
                cs_c[tid] = c; cs_s[tid] = sn;
                log[(size_t)round * h + tid] = make_double2(c, sn);
            }
            __syncthreads();
            // S_AB <- J_A^T S_AB J_B with J = [[c, s], [-s, c]] on the (p, q) plane
            for (int A = tid >> 5; A < h; A += nt >> 5) {
                const int p = pr_p[A] * m, q = pr_q[A] * m;
                const double ca = cs_c[A], sa = cs_s[A];
                for (int B = tid & 31; B < h; B += 32) {
                    const int u = pr_p[B], v = pr_q[B];
                    const double cb = cs_c[B], sb = cs_s[B];
                    const double spu = S[p + u], spv = S[p + v];
                    const double squ = S[q + u], sqv = S[q + v];
                    const double rpu = ca * spu - sa * squ, rpv = ca * spv - sa * sqv;
                    const double rqu = sa * spu + ca * squ, rqv = sa * spv + ca * sqv;
                    S[p + u] = cb * rpu - sb * rpv;
                    S[p + v] = sb * rpu + cb * rpv;
                    S[q + u] = cb * rqu - sb * rqv;
                    S[q + v] = sb * rqu + cb * rqv;
                }
            }
            __syncthreads();
        }
        if (s_rot == 0) { ++sweep; break; }
        __syncthreads();
    }
    // order by descending eigenvalue (rank sort; ties by index)
    for (int i = tid; i < m; i += nt) s_diag[i] = S[i * m + i];
    __syncthreads();
    for (int j = tid; j < m; j += nt) {
        int rk = 0;
        const double x = s_diag[j];
        for (int i = 0; i < m; ++i) rk += (s_diag[i] > x) || (s_diag[i] == x && i < j);
        head[1 + j] = rk;
        theta[rk] = x;
    }
    if (tid == 0) {
        head[0] = round;
        if (sweeps_out) *sweeps_out = (double)sweep;
    }
}

// W = product of the logged rotations, columns permuted to descending eigenvalue order.  A warp owns
// a row of W (initially a unit vector) in shared memory and applies the rounds in order -- the
// rotations of one round touch disjoint column pairs, one or more per lane; the (c, s) of eight
// rounds at a time are staged in shared memory for the CTA's eight rows, the next chunk's loads in
// flight while the current one is applied.
constexpr int kApplyWarps = 8, kApplyChunk = 8;
__global__ void __launch_bounds__(kApplyWarps * 32)
apply_rotations_kernel(const int *head, const double2 *log, double *Wout, int m) {
    __shared__ double rows[kApplyWarps][kJacobiLogRitz];
    __shared__ double2 cs[2][kApplyChunk][kJacobiLogRitz / 2];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, h = m / 2;
    const int row = blockIdx.x * kApplyWarps + warp;
    for (int j = lane; j < m; j += 32) rows[warp][j] = (j == row) ? 1.0 : 0.0;
    const int nrounds = head[0];
    const int nchunks = (nrounds + kApplyChunk - 1) / kApplyChunk;
    constexpr int kPre = (kApplyChunk * (kJacobiLogRitz / 2) + kApplyWarps * 32 - 1) / (kApplyWarps * 32);
    double2 pre[kPre];
    auto fetch = [&](int ch) {
#pragma unroll
        for (int i = 0; i < kPre; ++i) {
            const int e = tid + i * kApplyWarps * 32;
            const int R = ch * kApplyChunk + e / h;
            pre[i] = (e < kApplyChunk * h && R < nrounds) ? log[(size_t)R * h + e % h] : make_double2(1.0, 0.0);
        }
    };
    auto stash = [&](int buf) {
#pragma unroll
        for (int i = 0; i < kPre; ++i) {
            const int e = tid + i * kApplyWarps * 32;
            if (e < kApplyChunk * h) cs[buf][e / h][e % h] = pre[i];
        }
    };
    if (nchunks > 0) { fetch(0); stash(0); }
    __syncthreads();
    // the pairs of this lane's B = lane, lane + 32, ...: p = (r + B) mod (m - 1) and q = (r - B) mod (m - 1)
    // both step up by one from a round to the next (pair 0 keeps p = m - 1), so no round needs a division
    constexpr int kPairs = (kJacobiLogRitz / 2 + 31) / 32;
    int pp[kPairs], qq[kPairs];
#pragma unroll
    for (int i = 0; i < kPairs; ++i) {
        const int B = lane + 32 * i;
        pp[i] = B == 0 ? m - 1 : B % (m - 1);
        qq[i] = B == 0 ? 0 : (m - 1 - B % (m - 1)) % (m - 1);
    }
    for (int ch = 0; ch < nchunks; ++ch) {
        if (ch + 1 < nchunks) fetch(ch + 1);
        double *w = rows[warp];
        for (int t = 0; t < kApplyChunk && ch * kApplyChunk + t < nrounds; ++t) {
#pragma unroll
            for (int i = 0; i < kPairs; ++i) {
                const int B = lane + 32 * i;
                if (B < h) {
                    const int u = min(pp[i], qq[i]), v = max(pp[i], qq[i]);
                    const double2 f = cs[ch & 1][t][B];
                    const double wu = w[u], wv = w[v];
                    w[u] = f.x * wu - f.y * wv;
                    w[v] = f.y * wu + f.x * wv;
                }
                if (B != 0) pp[i] = pp[i] + 1 == m - 1 ? 0 : pp[i] + 1;
                qq[i] = qq[i] + 1 == m - 1 ? 0 : qq[i] + 1;
            }
            __syncwarp();
        }
        if (ch + 1 < nchunks) stash((ch + 1) & 1);
        __syncthreads();
    }
    if (row < m)
        for (int j = lane; j < m; j += 32) Wout[(int64_t)row * m + head[1 + j]] = rows[warp][j];
}

// ---------------------------------------------------------------------------------------
// Polynomial filter of the subspace iteration (Chebyshev-filtered subspace iteration).
// With the unwanted part of the spectrum inside [0, b], b = the smallest Ritz value of the block,
// and c = e = b / 2:
//   degree 1   Y1 = (G - c) Q / e                 a shifted power step: the k-th wanted direction
//              gains 2 lambda_k / b - 1 on the unwanted ones, where a plain step gains lambda_k / b;
//   degree 2   Y2 = T_2((G - c) / e) Q = 2 (G - c) Y1 / e - Q: for the configured power-law spectra
//              ~10 per two multiplications by G, where two plain steps gain ~2.8.
// The coefficients come from the Ritz values on the device.  Degree 2 lifts the leading direction
// over the k-th one by ~(lambda_1 / lambda_k)^2 per iteration; the orthonormalisation that follows
// works in fp64 and needs the columns to stay independent, so the host asks for it only while
// that ratio stays below 1e12 (filter_safe_kernel).  When b is not positive against theta_1 (a
// block wider than the rank of G) the step is a plain power step.
// ---------------------------------------------------------------------------------------
struct FilterCoef {
    double a1, b1, a2, b2, g2;   // Y1 = a1 (G Q) + b1 Q,  Y2 = a2 (G Y1) + b2 Y1 + g2 Q
    int deg2_safe;
};
__device__ __forceinline__ FilterCoef filter_coef(const double *theta, int m, int k) {
    const double t1 = theta[0], tk = theta[k - 1], b = theta[m - 1];
    FilterCoef f;
    const bool shift = isfinite(t1) && isfinite(b) && t1 > 0.0 && b > 1e-12 * t1;
    if (shift) {
        const double e = 0.5 * b;
        const double x1 = (t1 - e) / e, xk = (tk - e) / e;
        const double g1 = 2.0 * x1 * x1 - 1.0, gk = fabs(2.0 * xk * xk - 1.0);
        f.deg2_safe = g1 <= 1e12 * fmax(gk, 1.0) ? 1 : 0;
        f.a1 = 1.0 / e; f.b1 = -1.0;          // (Z - c Q) / e with c = e
        f.a2 = 2.0 / e; f.b2 = -2.0; f.g2 = -1.0;
    } else {
        f.deg2_safe = 0;
        f.a1 = (isfinite(t1) && t1 > 0.0) ? 1.0 / t1 : 1.0;
        f.b1 = 0.0;
        f.a2 = f.a1; f.b2 = 0.0; f.g2 = 0.0;   // (never used: the host takes degree 1 when deg2_safe is 0)
    }
    return f;
}
__global__ void filter_safe_kernel(const double *theta, int m, int k, double *flag) {
    *flag = (double)filter_coef(theta, m, k).deg2_safe;
}
// Y1 <- a1 Y1 + b1 Q   (Y1 holds G Q on entry)
__global__ void filter_first_kernel(double *Y1, const double *Q, const double *theta, int m, int k, int64_t n) {
    const FilterCoef f = filter_coef(theta, m, k);
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x)
        Y1[e] = f.a1 * Y1[e] + f.b1 * Q[e];
}
// Y2 <- a2 Y2 + b2 Y1 + g2 Q   (Y2 holds G Y1 on entry)
__global__ void filter_second_kernel(double *Y2, const double *Y1, const double *Q, const double *theta, int m, int k,
                                     int64_t n) {
    const FilterCoef f = filter_coef(theta, m, k);
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x)
        Y2[e] = f.a2 * Y2[e] + f.b2 * Y1[e] + f.g2 * Q[e];
}

// resid[j] = | Z[:, j] - theta[j] Q[:, j] |_2  for j < k;  one CTA per column
__global__ void residual_kernel(const double *Z, const double *Q, const double *theta, int D, int m,
                                double *resid) {
    __shared__ double red[256];
    const int j = blockIdx.x;
    const double th = theta[j];
    double s = 0.0;
    for (int i = threadIdx.x; i < D; i += 256) {
        const double r = Z[(int64_t)i * m + j] - th * Q[(int64_t)i * m + j];
        s += r * r;
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
        __syncthreads();
    }
    if (threadIdx.x == 0) resid[j] = sqrt(red[0]);
}

// scal[1] = max_j resid[j] / max(theta[0], tiny)
__global__ void max_residual_kernel(const double *resid, const double *theta, int k, double *scal) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        double mx = 0.0;
        for (int j = 0; j < k; ++j) mx = fmax(mx, resid[j]);
        const double t0 = fabs(theta[0]);
        scal[1] = (t0 > 0.0) ? mx / t0 : 0.0;
    }
}

// V_k (fp32) <- first k columns of Q with the sign convention; lambda <- theta[:k]
__global__ void emit_basis_kernel(const double *Q, const double *theta, int D, int m, int k, float *Vk,
                                  double *lambda) {
    __shared__ double best_abs[256];
    __shared__ double best_val[256];
    const int j = blockIdx.x;
    double ba = -1.0, bv = 0.0;
    for (int i = threadIdx.x; i < D; i += 256) {   // first index of the largest magnitude
        const double v = Q[(int64_t)i * m + j];
        if (fabs(v) > ba) { ba = fabs(v); bv = v; }
    }
    best_abs[threadIdx.x] = ba;
    best_val[threadIdx.x] = bv;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if (threadIdx.x < w && best_abs[threadIdx.x + w] > best_abs[threadIdx.x]) {
            best_abs[threadIdx.x] = best_abs[threadIdx.x + w];
            best_val[threadIdx.x] = best_val[threadIdx.x + w];
        }
        __syncthreads();
    }
    const double sgn = (best_val[0] < 0.0) ? -1.0 : 1.0;
    for (int i = threadIdx.x; i < D; i += 256) Vk[(int64_t)i * k + j] = (float)(sgn * Q[(int64_t)i * m + j]);
    if (threadIdx.x == 0 && lambda) lambda[j] = theta[j];
}

__global__ void copy_scalar_kernel(const double *src, double *dst) { *dst = *src; }


}  // namespace

size_t calib_workspace_bytes(int D, int k) { return calib_layout(D, k).total; }

int calib_begin(int D, int k, void *ws, cudaStream_t s) {
    const CalibLayout L = calib_layout(D, k);
    char *w = (char *)ws;
    init_header_kernel<<<1, 1, 0, s>>>((CalibHeader *)w, D, k);
    zero_kernel<<<grid_for((int64_t)D * D), 256, 0, s>>>((double *)(w + L.G), (int64_t)D * D);
    count_launch(2);
    return check_last_launch();
}

size_t calib_gram_offset() { return kHeaderBytes; }

int calib_accumulate(const void *F, int64_t M, int D, int64_t ld, int dtype, void *ws, cudaStream_t s) {
    // G sits at a fixed offset whatever k is
    char *w = (char *)ws;
    double *G = (double *)(w + kHeaderBytes);
    int rc;
    if (umma_gram_supported(M, D, ld, dtype)) {
        const CalibLayout L = calib_layout(D, 8);
        double *scratch = umma_gram_scratch_bytes(D) ? (double *)(w + L.gram_scratch) : nullptr;
        rc = umma_gram_accumulate(F, M, D, ld, G, scratch, &reinterpret_cast<CalibHeader *>(w)->status, s);
    } else if (dtype == SVDCACHE_BF16) {
        const __nv_bfloat16 *f = (const __nv_bfloat16 *)F;
        rc = dgemm<__nv_bfloat16, __nv_bfloat16, true>(f, ld, f, ld, G, D, D, D, M, true, true, s);
    } else {
        const float *f = (const float *)F;
        rc = dgemm<float, float, true>(f, ld, f, ld, G, D, D, D, M, true, true, s);
    }
    if (rc) return rc;
    add_rows_kernel<<<1, 1, 0, s>>>((CalibHeader *)w, M, D);
    count_launch();
    return check_last_launch();
}

namespace {

// Q (D x m) <- orthonormal basis of the columns of Zin (scaled Cholesky-QR, twice; columns
// found dependent in the first pass are re-seeded before the second).  Zin is destroyed;
// T is scratch.  The result ends up in Zin's buffer, returned through *out.
int orthonormalize(double *Zin, double *T, double *S, double *X, int *dead, int D, int m, uint64_t salt,
                   double **out, cudaStream_t s, Partials ps) {
    double *src = Zin, *dst = T;
    for (int pass = 0; pass < 2; ++pass) {
        int rc = dgemm<double, double, true>(src, m, src, m, S, m, m, m, D, false, false, s, ps);
        if (rc) return rc;
        symmetrize_kernel<<<grid_for((int64_t)m * m), 256, 0, s>>>(S, m, 1);
        if (m <= kCholSmemRitz) {
            const size_t cb = (size_t)m * (m + 1) * 8;
            if (cb > 40 * 1024) {   // per call: the attribute belongs to the current device's copy of the kernel
                rc = record_cuda(cudaFuncSetAttribute(chol_inv_smem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cb));
                if (rc) return rc;
            }
            chol_inv_smem_kernel<<<1, 1024, cb, s>>>(S, X, m, dead);
        } else {
            chol_inv_kernel<<<1, 1024, 0, s>>>(S, X, m, dead);
        }
        count_launch(2);
        rc = dgemm<double, double, false>(src, m, X, m, dst, m, D, m, m, false, false, s);
        if (rc) return rc;
        if (pass == 0) {
            reseed_dead_kernel<<<grid_for((int64_t)D * m), 256, 0, s>>>(dst, D, m, dead, salt);
            count_launch();
        }
        std::swap(src, dst);
    }
    *out = src;
    return check_last_launch();
}

}  // namespace

int calib_finish(int D, int k, float *Vk, double *lambda, double *trace, double *info, void *ws,
                 cudaStream_t s) {
    const CalibLayout L = calib_layout(D, k);
    const int m = L.m;
    if (m > kMaxRitz || (m % 2) != 0) return SVDCACHE_ERR_BAD_SHAPE;
    char *w = (char *)ws;
    double *G = (double *)(w + L.G);
    double *bufA = (double *)(w + L.Q), *bufB = (double *)(w + L.Z), *bufC = (double *)(w + L.T);
    double *S = (double *)(w + L.S), *W = (double *)(w + L.W), *X = (double *)(w + L.X);
    double *theta = (double *)(w + L.theta), *resid = (double *)(w + L.resid), *scal = (double *)(w + L.scal);
    // scal[0] = trace, scal[1] = max relative residual, scal[2] = Jacobi sweeps

    int rc;
    // an accumulation kernel whose bounded wait ran out has left its error in the header
    {
        CalibHeader h;
        rc = record_cuda(cudaMemcpyAsync(&h, w, sizeof(h), cudaMemcpyDeviceToHost, s));
        if (rc) return rc;
        rc = record_cuda(cudaStreamSynchronize(s));
        if (rc) return rc;
        if (h.status != SVDCACHE_OK) return h.status;
        // the workspace must be the one svdcache_calibrate_begin laid out for this width, and for a
        // rank at least as large (G sits at a fixed offset; the solver's buffers grow with k)
        if (h.D != D || k > h.k_max) return SVDCACHE_ERR_WORKSPACE;
    }

    symmetrize_kernel<<<grid_for((int64_t)D * D), 256, 0, s>>>(G, D, 0);
    trace_kernel<<<1, 256, 0, s>>>(G, D, scal);
    init_block_kernel<<<grid_for((int64_t)D * m), 256, 0, s>>>(bufA, (int64_t)D * m);
    count_launch(3);
    rc = check_last_launch();
    if (rc) return rc;


    int *dead = (int *)(w + L.dead);
    double *Q = nullptr;
    const Partials ps{(double *)(w + L.partials), L.partial_bytes};
    rc = orthonormalize(bufA, bufB, S, X, dead, D, m, 1, &Q, s, ps);
    if (rc) return rc;
    auto others = [&](double *q, double **z, double **t) {
        double *all[3] = {bufA, bufB, bufC};
        int n = 0;
        double *o[2];
        for (double *b : all)
            if (b != q) o[n++] = b;
        *z = o[0]; *t = o[1];
    };

    // One iteration: Z = G Q; on a Ritz iteration Rayleigh-Ritz on span(Q) (S = Q^T Z = W Theta W^T,
    // Q <- Q W, Z <- Z W: no further product with G) and the residual check; then the polynomial
    // filter on top of Z (degree 2: one more product with G) and Q <- orthonormalise(filtered block).
    // The Rayleigh-Ritz step (the m x m eigen-problem is the serial, single-CTA part) runs on the
    // first iterations, which turn the random start block into ordered eigenvector estimates and
    // give the filter its bounds, and on every second one after that (every fourth with the
    // degree-1 filter); in between, the QR step takes out of every column its components along the
    // columns before it, so the columns stay ordered and nearly orthogonal and the scaled
    // Cholesky-QR stays well conditioned.
    const double tol = 1e-12;
    const int max_mult = 200;
    double max_rel = 1.0;
    int mult = 0, degree = 1;
    bool converged = false;
    const int64_t nelem = (int64_t)D * m;
    for (int iter = 1;; ++iter) {
        const bool last = mult + 4 > max_mult;   // no room for another whole iteration after this one
        double *Z, *T;
        others(Q, &Z, &T);
        rc = dgemm<double, double, true>(G, D, Q, m, Z, m, D, m, D, false, false, s, ps);   // Z = G Q
        if (rc) return rc;
        ++mult;
        const bool ritz_step = iter <= 3 || (degree == 2 ? (iter & 1) != 0 : (iter % 4) == 0) || last;
        double *block = Q, *image = Z, *spare = T;   // the filter acts on (block, G block); spare is free
        if (ritz_step) {
            rc = dgemm<double, double, true>(Q, m, Z, m, S, m, m, m, D, false, false, s, ps);   // S = Q^T Z
            if (rc) return rc;
            symmetrize_kernel<<<grid_for((int64_t)m * m), 256, 0, s>>>(S, m, 1);
            {
                const size_t jb = 2 * (size_t)m * m * 8;
                const bool fits = jb <= kJacobiSmemMax;
                // the rotation log borrows the split products' scratch, which is idle during the Ritz step
                const size_t log_bytes = kJacobiLogHead + (size_t)kJacobiMaxSweeps * (m - 1) * (m / 2) * sizeof(double2);
                if (m <= kJacobiLogRitz && ps.buf != nullptr && log_bytes <= ps.bytes) {
                    const size_t sb = (size_t)m * m * 8;
                    if (sb > 40 * 1024) {   // per call: the attribute belongs to the current device's copy of the kernel
                        rc = record_cuda(cudaFuncSetAttribute(jacobi_logged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sb));
                        if (rc) return rc;
                    }
                    int *head = (int *)ps.buf;
                    double2 *rot = (double2 *)((char *)ps.buf + kJacobiLogHead);
                    jacobi_logged_kernel<<<1, kJacobiThreads, sb, s>>>(S, theta, m, scal + 2, head, rot);
                    apply_rotations_kernel<<<(m + kApplyWarps - 1) / kApplyWarps, kApplyWarps * 32, 0, s>>>(head, rot, W, m);
                    count_launch();
                } else {
                    if (fits && jb > 40 * 1024) {   // per call: the attribute belongs to the current device's copy of the kernel
                        rc = record_cuda(cudaFuncSetAttribute(jacobi_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kJacobiSmemMax));
                        if (rc) return rc;
                    }
                    jacobi_kernel<<<1, kJacobiThreads, fits ? jb : 0, s>>>(S, X, W, theta, m, scal + 2, fits ? 1 : 0);
                }
            }
            count_launch(2);
            rc = dgemm<double, double, false>(Q, m, W, m, T, m, D, m, m, false, false, s);  // ritz = Q W
            if (rc) return rc;
            rc = dgemm<double, double, false>(Z, m, W, m, Q, m, D, m, m, false, false, s);  // image = Z W
            if (rc) return rc;
            block = T; image = Q; spare = Z;
            if (iter >= 2) {
                residual_kernel<<<k, 256, 0, s>>>(image, block, theta, D, m, resid);
                max_residual_kernel<<<1, 32, 0, s>>>(resid, theta, k, scal);
                count_launch(2);
            }
            filter_safe_kernel<<<1, 1, 0, s>>>(theta, m, k, scal + 3);
            count_launch();
            double back[3] = {1.0, 0.0, 0.0};   // scal[1..3]: max relative residual, Jacobi sweeps, degree-2 flag
            rc = record_cuda(cudaMemcpyAsync(back, scal + 1, sizeof(back), cudaMemcpyDeviceToHost, s));
            if (rc) return rc;
            rc = record_cuda(cudaStreamSynchronize(s));
            if (rc) return rc;
            degree = back[2] != 0.0 ? 2 : 1;
            if (iter >= 2) {
                max_rel = back[0];
                if (max_rel <= tol || last) {
                    converged = max_rel <= tol;
                    Q = block;
                    break;
                }
            }
        }
        filter_first_kernel<<<grid_for(nelem), 256, 0, s>>>(image, block, theta, m, k, nelem);           // Y1, in place
        count_launch();
        if (degree == 1) {
            rc = orthonormalize(image, spare, S, X, dead, D, m, (uint64_t)mult + 1, &Q, s, ps);
            if (rc) return rc;
            continue;
        }
        rc = dgemm<double, double, true>(G, D, image, m, spare, m, D, m, D, false, false, s, ps);       // G Y1
        if (rc) return rc;
        ++mult;
        filter_second_kernel<<<grid_for(nelem), 256, 0, s>>>(spare, image, block, theta, m, k, nelem);  // Y2, in place
        count_launch();
        rc = orthonormalize(spare, image, S, X, dead, D, m, (uint64_t)mult + 1, &Q, s, ps);
        if (rc) return rc;
    }

    emit_basis_kernel<<<k, 256, 0, s>>>(Q, theta, D, m, k, Vk, lambda);
    count_launch();
    if (trace) {
        copy_scalar_kernel<<<1, 1, 0, s>>>(scal, trace);
        count_launch();
    }
    rc = check_last_launch();
    if (rc) return rc;
    double sweeps = 0.0;
    rc = record_cuda(cudaMemcpyAsync(&sweeps, scal + 2, sizeof(double), cudaMemcpyDeviceToHost, s));
    if (rc) return rc;
    rc = record_cuda(cudaStreamSynchronize(s));
    if (rc) return rc;
    if (info) {
        info[0] = (double)mult;
        info[1] = max_rel;
        info[2] = (double)m;
        info[3] = sweeps;
    }
    return converged ? SVDCACHE_OK : SVDCACHE_ERR_NOT_CONVERGED;
}

}  // namespace svdc

// ---------------------------------------------------------------------------------------
// Calibration without a caller-supplied workspace: the scratch that carries G and the
// iteration blocks is a fixed array in the library's own device image.
// ---------------------------------------------------------------------------------------
namespace svdc {
namespace {

constexpr size_t kBuiltinScratchBytes = SVDCACHE_BUILTIN_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void *g_scratch_addr[kMaxDevices] = {};   // device address of g_builtin_scratch, per device ordinal

// In host code `g_builtin_scratch` only names the symbol; the address a kernel can use
// has to be asked for, once per device, with that device current.
int builtin_scratch(void **out) {
    int dev = -1;
    int rc = record_cuda(cudaGetDevice(&dev));
    if (rc) return rc;
    if (dev < 0 || dev >= kMaxDevices) return SVDCACHE_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        rc = record_cuda(cudaGetSymbolAddress(&ptr, g_builtin_scratch));
        if (rc) return rc;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return SVDCACHE_OK;
}

}  // namespace
}  // namespace svdc

extern "C" int svdcache_calibrate_noalloc(const void *Fstack, int64_t M, int D, int64_t ld, int dtype, int k,
                                          float *Vk, double *lambda, double *trace, double *info, void *stream) {
    using namespace svdc;
    if (dtype != SVDCACHE_F32 && dtype != SVDCACHE_BF16) return SVDCACHE_ERR_INVALID_ARG;
    if (M < 1 || D < 8 || D > 16384 || (D % 8) != 0) return SVDCACHE_ERR_BAD_SHAPE;
    if (k < 8 || k > 256 || (k % 8) != 0 || k > D) return SVDCACHE_ERR_BAD_SHAPE;
    if (!Fstack || !Vk) return SVDCACHE_ERR_INVALID_ARG;
    if (ld < D) return SVDCACHE_ERR_BAD_SHAPE;
    if (((size_t)ld * elem_bytes(dtype)) % 16 != 0) return SVDCACHE_ERR_BAD_ALIGN;
    if ((reinterpret_cast<uintptr_t>(Fstack) & 15u) || (reinterpret_cast<uintptr_t>(Vk) & 15u)) return SVDCACHE_ERR_BAD_ALIGN;
    if (calib_workspace_bytes(D, k) > kBuiltinScratchBytes) return SVDCACHE_ERR_SCRATCH_LIMIT;
    void *ws = nullptr;
    int rc = builtin_scratch(&ws);
    if (rc) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    rc = calib_begin(D, k, ws, s);   // clears the header and G: nothing of the previous call is reused
    if (rc) return rc;
    rc = calib_accumulate(Fstack, M, D, ld, dtype, ws, s);
    if (rc) return rc;
    return calib_finish(D, k, Vk, lambda, trace, info, ws, s);
}

