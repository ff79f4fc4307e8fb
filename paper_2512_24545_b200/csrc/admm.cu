// ADMM refinement of one MDBF factor with the other held fixed (Section "ADMM Refinement"):
//
//     U_tilde = (W V + rho (U - Lam)) (V^T V + rho I)^-1        Eq. admm-U-tilde
//     U       = MSVID_l[U_tilde + Lam]                          Eq. admm-U-prox
//     Lam     = Lam + U_tilde - U                               Eq. admm-U-dual
//
// W is N x M, V is M x R, U and Lam are N x R (dense values of the factor), all fp32 row-major on the device.  The
// update of the other factor is the same call on the transposed problem (transpose_w).
//
// The two dense products (W V and V^T V, once per call) run on the tensor cores at close to fp32 accuracy (gemm3x.cu: TF32
// operands in a three-term split); V's operand images serve both, as the right operand of W V and as both operands of
// V^T V.  The Cholesky factorisation of the R x R system (cuSOLVER) and one triangular solve for the factor's inverse
// (cuBLAS) are library routines; the inverse of the system is formed and then applied, in every inner iteration, by the
// same tensor-core product.  Everything
// specific to the method is this library's own: the MSVID step (mdbf_msvid: sign mask + rank-l envelope on the tensor
// cores), the elementwise passes around it, and the reconstruction of the dense factor from the compact one fused with
// the dual update.
//
// The system is symmetric, so the column-major solver works on the row-major memory as it is; what it calls the lower
// triangle are the rows above the diagonal here.
#include <cublas_v2.h>
#include <cusolverDn.h>

#include <algorithm>
#include <cstdint>

#include "common.cuh"

namespace mdbf {
namespace admm {

struct Libs {
    cublasHandle_t blas = nullptr;
    cusolverDnHandle_t solver = nullptr;
    float *potrf_ws = nullptr;          // the factorisation's scratch, as large as the largest request so far
    int potrf_floats = 0;
    int device = -1;
    cudaStream_t side = nullptr;        // the R x R system is factored and inverted here while W V runs on the caller's stream
    cudaEvent_t fork = nullptr, join = nullptr;
};
static thread_local Libs g_libs;

static mdbf_status_t get_libs(int device, cudaStream_t st, Libs **out) {
    Libs &L = g_libs;
    if (L.device != device) {
        if (L.blas) cublasDestroy(L.blas);
        if (L.solver) cusolverDnDestroy(L.solver);
        if (L.potrf_ws) cudaFree(L.potrf_ws);
        if (L.side) cudaStreamDestroy(L.side);
        if (L.fork) cudaEventDestroy(L.fork);
        if (L.join) cudaEventDestroy(L.join);
        L = Libs();
        if (cublasCreate(&L.blas) != CUBLAS_STATUS_SUCCESS) { L = Libs(); set_error("cublasCreate failed"); return MDBF_ERR_CUDA; }
        if (cusolverDnCreate(&L.solver) != CUSOLVER_STATUS_SUCCESS) {
            cublasDestroy(L.blas);
            L = Libs();
            set_error("cusolverDnCreate failed");
            return MDBF_ERR_CUDA;
        }
        cublasSetMathMode(L.blas, CUBLAS_PEDANTIC_MATH);          // plain fp32 products
        if (cudaStreamCreateWithFlags(&L.side, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&L.fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&L.join, cudaEventDisableTiming) != cudaSuccess ||
            cublasSetStream(L.blas, L.side) != CUBLAS_STATUS_SUCCESS || cusolverDnSetStream(L.solver, L.side) != CUSOLVER_STATUS_SUCCESS) {
            cublasDestroy(L.blas);
            cusolverDnDestroy(L.solver);
            if (L.side) cudaStreamDestroy(L.side);
            if (L.fork) cudaEventDestroy(L.fork);
            if (L.join) cudaEventDestroy(L.join);
            L = Libs();
            set_error("could not create the side stream of the refinement step");
            return MDBF_ERR_CUDA;
        }
        L.device = device;
    }
    (void)st;
    *out = &L;
    return MDBF_OK;
}

// the solver's scratch, as large as the largest request so far
static mdbf_status_t grow_scratch(Libs *L, int floats, cudaStream_t st, const char *who) {
    if (floats <= L->potrf_floats) return MDBF_OK;
    MDBF_CUDA(cudaStreamSynchronize(st));                         // the stream that uses it: the old scratch may still be in use
    if (L->potrf_ws) cudaFree(L->potrf_ws);
    L->potrf_ws = nullptr;
    L->potrf_floats = 0;
    if (dev_malloc(&L->potrf_ws, (size_t)floats * sizeof(float)) != cudaSuccess) {
        set_error("%s: out of device memory for the solver's scratch (%zu bytes)", who, (size_t)floats * sizeof(float));
        return MDBF_ERR_CUDA;
    }
    L->potrf_floats = floats;
    return MDBF_OK;
}

__global__ void ridge_kernel(float *__restrict__ G, int r, float rho) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < r) G[(size_t)i * r + i] += rho;
}
__global__ void identity_kernel(float *__restrict__ X, int r) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x, a = blockIdx.y;
    if (b < r) X[(size_t)a * r + b] = a == b ? 1.f : 0.f;
}
// T = B0 + rho (U - Lam)
__global__ void rhs_kernel(const float *__restrict__ B0, const float *__restrict__ U, const float *__restrict__ Lam, float rho,
                           float *__restrict__ T, size_t count) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < count; e += (size_t)gridDim.x * blockDim.x)
        T[e] = B0[e] + rho * (U[e] - Lam[e]);
}
// Z = U_tilde + Lam
__global__ void sum_kernel(const float *__restrict__ Ut, const float *__restrict__ Lam, float *__restrict__ Z, size_t count) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < count; e += (size_t)gridDim.x * blockDim.x) Z[e] = Ut[e] + Lam[e];
}
// U = S (.) (Ul Vl^T) entry by entry from the compact MSVID result, and Lam += U_tilde - U.
// CTA = 32 rows x 256 columns; thread = column (its row of Vl in registers), the rows' Ul in shared memory.
constexpr int RC_ROWS = 32, RC_COLS = 256, RC_MAXL = 32;
__global__ void __launch_bounds__(RC_COLS) recon_dual_kernel(const uint32_t *__restrict__ S, const float *__restrict__ Ul,
                                                             const float *__restrict__ Vl, int l, const float *__restrict__ Ut,
                                                             float *__restrict__ U, float *__restrict__ Lam, int n, int r, int nwords) {
    __shared__ float us[RC_ROWS][RC_MAXL];
    const int i0 = blockIdx.y * RC_ROWS;
    for (int e = threadIdx.x; e < RC_ROWS * RC_MAXL; e += RC_COLS) {
        const int i = e / RC_MAXL, t = e - i * RC_MAXL;
        us[i][t] = (i0 + i < n && t < l) ? Ul[(size_t)(i0 + i) * l + t] : 0.f;
    }
    __syncthreads();
    const int j = blockIdx.x * RC_COLS + threadIdx.x;
    if (j >= r) return;
    float v[RC_MAXL];
#pragma unroll
    for (int t = 0; t < RC_MAXL; ++t) v[t] = t < l ? Vl[(size_t)j * l + t] : 0.f;
    for (int ib = 0; ib < RC_ROWS && i0 + ib < n; ib += 4) {     // four rows at a time: their loads are in flight together
        float ut[4], lm[4];
        uint32_t word[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const bool in = i0 + ib + u < n;
            const size_t at = (size_t)(i0 + ib + u) * r + j;
            ut[u] = in ? Ut[at] : 0.f;
            lm[u] = in ? Lam[at] : 0.f;
            word[u] = in ? S[(size_t)(i0 + ib + u) * nwords + (j >> 5)] : 0u;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (i0 + ib + u >= n) break;
            float e = 0.f;
#pragma unroll
            for (int t = 0; t < RC_MAXL; ++t) e = fmaf(us[ib + u][t], v[t], e);
            const float val = ((word[u] >> (j & 31)) & 1u) ? -e : e;
            const size_t at = (size_t)(i0 + ib + u) * r + j;
            U[at] = val;
            Lam[at] = lm[u] + (ut[u] - val);
        }
    }
}
// a failed factorisation (not expected: the system is positive definite for rho > 0) or an expired wait of the product
// kernel turns the singular values into NaN
__global__ void flag_kernel(const int *__restrict__ info, float *__restrict__ sigma, int l) {
    if ((info[0] != 0 || info[2] != 0) && threadIdx.x < l) sigma[threadIdx.x] = __int_as_float(0x7fc00000);
}

static size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }
struct Scratch {
    float *B0, *T, *Z, *G;
    uint32_t *Wimg, *Vimg;      // operand images of op(W) (N row tiles, M deep) and of V^T (R row tiles, M deep)
    uint32_t *Yimg;             // images of L^-T (R x R), formed on the side stream while W's are in use
    int *info;                  // [0], [1]: the solver's; [2]: status word of the product kernel
    char *msvid;
    size_t msvid_bytes;
};
static mdbf_status_t carve(Scratch *w, char *base, int64_t n, int64_t m, int64_t r, int32_t l, size_t *total) {
    size_t msv = 0;
    mdbf_status_t rc = mdbf_msvid_workspace_bytes(n, r, l, &msv);
    if (rc) return rc;
    size_t off = 0;
    auto take = [&](size_t bytes) { char *p = base ? base + off : nullptr; off += align256(bytes); return p; };
    float *B0 = (float *)take((size_t)n * r * sizeof(float));
    float *T = (float *)take((size_t)n * r * sizeof(float));
    float *Z = (float *)take((size_t)n * r * sizeof(float));
    float *G = (float *)take((size_t)r * r * sizeof(float));
    uint32_t *Wimg = (uint32_t *)take(gemm3x_image_bytes(n, m));
    uint32_t *Vimg = (uint32_t *)take(gemm3x_image_bytes(r, m));
    uint32_t *Yimg = (uint32_t *)take(gemm3x_image_bytes(r, r));
    int *info = (int *)take(4 * sizeof(int));
    char *mw = take(msv);
    if (w) { w->B0 = B0; w->T = T; w->Z = Z; w->G = G; w->Wimg = Wimg; w->Vimg = Vimg; w->Yimg = Yimg; w->info = info; w->msvid = mw; w->msvid_bytes = msv; }
    *total = off;
    return MDBF_OK;
}
static mdbf_status_t check_shape(const char *who, int64_t n, int64_t m, int64_t r, int32_t l) {
    if (n < 1 || m < 1 || r < 1 || n > (1 << 21) || m > (1 << 21) || r > 32768 || n * r > (1LL << 31) - 1 || n * m > (1LL << 40)) {   // grid limits of the tiled kernels
        set_error("%s: sizes N=%lld M=%lld R=%lld outside the supported range", who, (long long)n, (long long)m, (long long)r);
        return MDBF_ERR_SHAPE;
    }
    if (r > n || r > m) {
        set_error("%s: the inner dimension R=%lld exceeds min(N, M) = min(%lld, %lld)", who, (long long)r, (long long)n, (long long)m);
        return MDBF_ERR_SHAPE;
    }
    if (l < 1 || l > kMaxL || l > n || l > r) {
        set_error("%s: l=%d outside [1, min(%d, N, R)]", who, l, kMaxL);
        return MDBF_ERR_SHAPE;
    }
    return MDBF_OK;
}

}  // namespace admm
}  // namespace mdbf

using namespace mdbf;

extern "C" mdbf_status_t mdbf_admm_workspace_bytes(int64_t n, int64_t m, int64_t r, int32_t l, size_t *bytes) {
    if (!bytes) { set_error("mdbf_admm_workspace_bytes: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    mdbf_status_t rc = admm::check_shape("mdbf_admm_workspace_bytes", n, m, r, l);
    if (rc) return rc;
    return admm::carve(nullptr, nullptr, n, m, r, l, bytes);
}

extern "C" mdbf_status_t mdbf_admm_factor_update(const float *W, int64_t w_rows, int64_t w_cols, int32_t transpose_w, const float *V,
                                                 int64_t r, float *U, float *Lambda, float rho, int32_t l, int32_t n_inner,
                                                 int32_t n_iter, const float *Q0, uint32_t *S_packed, float *Ul, float *Vl,
                                                 float *sigma, float *U_tilde, void *workspace, size_t workspace_bytes, void *stream) {
    const char *who = "mdbf_admm_factor_update";
    if (!W || !V || !U || !Lambda || !Q0 || !S_packed || !Ul || !Vl || !sigma || !workspace) {
        set_error("%s: NULL pointer", who);
        return MDBF_ERR_INVALID_ARG;
    }
    const int64_t n = transpose_w ? w_cols : w_rows, m = transpose_w ? w_rows : w_cols;
    mdbf_status_t rc = admm::check_shape(who, n, m, r, l);
    if (rc) return rc;
    if (!(rho > 0.f) || n_inner < 1 || n_inner > 1000 || n_iter < 1 || n_iter > 1000) {
        set_error("%s: rho=%g must be positive, n_inner=%d and n_iter=%d in [1, 1000]", who, (double)rho, n_inner, n_iter);
        return MDBF_ERR_INVALID_ARG;
    }
    admm::Scratch w;
    size_t need = 0;
    rc = admm::carve(&w, (char *)workspace, n, m, r, l, &need);
    if (rc) return rc;
    if (workspace_bytes < need || ((uintptr_t)workspace & 255u) != 0) {
        set_error("%s: the workspace must hold %zu bytes (mdbf_admm_workspace_bytes) on a 256-byte boundary; got %zu at %p", who, need,
                  workspace_bytes, workspace);
        return MDBF_ERR_INVALID_ARG;
    }
    int device = 0;
    rc = require_device(&device);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    admm::Libs *L = nullptr;
    rc = admm::get_libs(device, st, &L);
    if (rc) return rc;
    const int ni = (int)n, mi = (int)m, ri = (int)r;
    MDBF_CUDA(cudaMemsetAsync(w.info, 0, 4 * sizeof(int), st));
    // images: op(W)[i][k] = W[i * w_cols + k], or W[k * w_cols + i] when transposed;  V^T[j][k] = V[k * r + j]
    rc = gemm3x_split(V, 1, (size_t)r, ri, mi, w.Vimg, st);
    if (rc) return rc;
    // Fork.  Side stream: G = V^T V + rho I, its Cholesky factor, L X = I by one triangular solve (X = L^-1, column-major;
    // read row-major it is Y = L^-T), G^-1 = Y Y^T as a product of Y's images with themselves - the inverse written out,
    // as Eq. admm-U-tilde has it, so that every inner iteration's solve is one product on the tensor cores instead of two
    // triangular solves with N right-hand sides on the FP32 pipe.  Caller's stream meanwhile: W's images and B0 = op(W) V,
    // on all SMs but a few that are left to the solver's small kernels.  Z is free until the loop below.
    cudaStream_t s2 = L->side;
    MDBF_CUDA(cudaEventRecord(L->fork, st));
    MDBF_CUDA(cudaStreamWaitEvent(s2, L->fork, 0));
    rc = gemm3x_run(w.Vimg, w.Vimg, w.G, ri, ri, mi, w.info + 2, s2);
    if (rc) return rc;
    admm::ridge_kernel<<<ceil_div(ri, 256), 256, 0, s2>>>(w.G, ri, rho);
    int lwork = 0;
    cusolverStatus_t ss = cusolverDnSpotrf_bufferSize(L->solver, CUBLAS_FILL_MODE_LOWER, ri, w.G, ri, &lwork);
    if (ss != CUSOLVER_STATUS_SUCCESS) { set_error("%s: cusolverDnSpotrf_bufferSize returned %d", who, (int)ss); return MDBF_ERR_CUDA; }
    rc = admm::grow_scratch(L, lwork, s2, who);
    if (rc) return rc;
    ss = cusolverDnSpotrf(L->solver, CUBLAS_FILL_MODE_LOWER, ri, w.G, ri, L->potrf_ws, L->potrf_floats, w.info);
    if (ss != CUSOLVER_STATUS_SUCCESS) { set_error("%s: cusolverDnSpotrf returned %d", who, (int)ss); return MDBF_ERR_CUDA; }
    admm::identity_kernel<<<dim3(ceil_div(ri, 256), ri), 256, 0, s2>>>(w.Z, ri);
    const float one = 1.f;
    cublasStatus_t bs = cublasStrsm(L->blas, CUBLAS_SIDE_LEFT, CUBLAS_FILL_MODE_LOWER, CUBLAS_OP_N, CUBLAS_DIAG_NON_UNIT, ri, ri, &one,
                                    w.G, ri, w.Z, ri);
    if (bs != CUBLAS_STATUS_SUCCESS) { set_error("%s: cublasStrsm returned %d", who, (int)bs); return MDBF_ERR_CUDA; }
    rc = gemm3x_split(w.Z, (size_t)r, 1, ri, ri, w.Yimg, s2);
    if (rc == MDBF_OK) rc = gemm3x_run(w.Yimg, w.Yimg, w.G, ri, ri, ri, w.info + 2, s2);
    if (rc) return rc;
    MDBF_CUDA(cudaEventRecord(L->join, s2));
    rc = transpose_w ? gemm3x_split(W, 1, (size_t)w_cols, ni, mi, w.Wimg, st) : gemm3x_split(W, (size_t)w_cols, 1, ni, mi, w.Wimg, st);
    if (rc == MDBF_OK) rc = gemm3x_run(w.Wimg, w.Vimg, w.B0, ni, ri, mi, w.info + 2, st, 24);
    if (rc) return rc;
    // Join; the inverse's images go where V's were (symmetric: rows serve as columns)
    MDBF_CUDA(cudaStreamWaitEvent(st, L->join, 0));
    rc = gemm3x_split(w.G, (size_t)r, 1, ri, ri, w.Vimg, st);
    if (rc) return rc;
    const size_t count = (size_t)n * r;
    const int ew_grid = (int)std::min<size_t>((count + 255) / 256, 148u * 16);
    const int nwords = (int)((r + 31) / 32);
    for (int it = 0; it < n_inner; ++it) {
        admm::rhs_kernel<<<ew_grid, 256, 0, st>>>(w.B0, U, Lambda, rho, w.T, count);
        // U_tilde = T G^-1, over T's own memory (its images live where W's were)
        rc = gemm3x_split(w.T, (size_t)r, 1, ni, ri, w.Wimg, st);
        if (rc == MDBF_OK) rc = gemm3x_run(w.Wimg, w.Vimg, w.T, ni, ri, ri, w.info + 2, st);
        if (rc) return rc;
        admm::sum_kernel<<<ew_grid, 256, 0, st>>>(w.T, Lambda, w.Z, count);
        rc = mdbf_msvid(w.Z, n, r, l, n_iter, Q0, S_packed, Ul, Vl, sigma, w.msvid, w.msvid_bytes, stream);
        if (rc) return rc;
        admm::recon_dual_kernel<<<dim3(ceil_div(ri, admm::RC_COLS), ceil_div(ni, admm::RC_ROWS)), admm::RC_COLS, 0, st>>>(
            S_packed, Ul, Vl, l, w.T, U, Lambda, ni, ri, nwords);
    }
    if (U_tilde) MDBF_CUDA(cudaMemcpyAsync(U_tilde, w.T, count * sizeof(float), cudaMemcpyDeviceToDevice, st));
    admm::flag_kernel<<<1, 32, 0, st>>>(w.info, sigma, l);                      // the factorisation's flag or an expired wait
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}
