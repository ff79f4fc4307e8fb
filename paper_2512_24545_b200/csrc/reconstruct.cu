// Dense W_hat = (S_A (.) U_A V_A^T)(S_B (.) U_B V_B^T)  (Eq. me-dbf-basis).
// Check path: factor tiles are formed element-wise from the packed signs and
// the stored envelopes and multiplied with fp64 accumulation, so the fp32
// result carries one rounding.
#include "common.cuh"

namespace mdbf {

constexpr int RT = 64;   // output tile (rows and columns)
constexpr int RJ = 16;   // inner-rank chunk

__global__ void __launch_bounds__(256)
reconstruct_kernel(const SignView wA, const SignView wB,
                   const void *__restrict__ UA, const void *__restrict__ VA,
                   const void *__restrict__ UB, const void *__restrict__ VB,
                   int d_out, int d_in, int k, int l, int env_dtype, float *__restrict__ W) {
    __shared__ double sU[RJ][RT + 1];   // U_hat[n, j] for the tile's rows, chunk of j
    __shared__ double sV[RJ][RT + 1];   // V_hat^T[j, i] for the tile's columns
    const int n0 = blockIdx.y * RT, i0 = blockIdx.x * RT;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    double acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;

    for (int j0 = 0; j0 < k; j0 += RJ) {
        // build the two factor tiles: RT*RJ entries each, 256 threads -> 4 entries per thread each
        for (int e = threadIdx.x; e < RT * RJ; e += 256) {
            {   // U_hat entry: row n = n0 + (e / RJ), column j = j0 + (e % RJ)
                const int rn = e / RJ, cj = e % RJ;
                const int n = n0 + rn, j = j0 + cj;
                double v = 0.0;
                if (n < d_out && j < k) {
                    for (int t = 0; t < l; ++t)
                        v += (double)env_load(UA, (size_t)n * l + t, env_dtype) *
                             (double)env_load(VA, (size_t)j * l + t, env_dtype);
                    if ((wA.word(n, j >> 5) >> (j & 31)) & 1u) v = -v;
                }
                sU[cj][rn] = v;
            }
            {   // V_hat^T entry: row j = j0 + (e / RT), column i = i0 + (e % RT)
                const int cj = e / RT, ci = e % RT;
                const int j = j0 + cj, i = i0 + ci;
                double v = 0.0;
                if (j < k && i < d_in) {
                    for (int s = 0; s < l; ++s)
                        v += (double)env_load(UB, (size_t)j * l + s, env_dtype) *
                             (double)env_load(VB, (size_t)i * l + s, env_dtype);
                    if ((wB.word(j, i >> 5) >> (i & 31)) & 1u) v = -v;
                }
                sV[cj][ci] = v;
            }
        }
        __syncthreads();
#pragma unroll
        for (int jj = 0; jj < RJ; ++jj) {
            double u[4], v[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) u[a] = sU[jj][ty * 4 + a];
#pragma unroll
            for (int b = 0; b < 4; ++b) v[b] = sV[jj][tx * 4 + b];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] += u[a] * v[b];
        }
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int n = n0 + ty * 4 + a;
        if (n >= d_out) continue;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int i = i0 + tx * 4 + b;
            if (i < d_in) W[(size_t)n * d_in + i] = (float)acc[a][b];
        }
    }
}

mdbf_status_t launch_reconstruct(const Layer &L, float *W, cudaStream_t st) {
    dim3 grid(ceil_div(L.d.d_in, RT), ceil_div(L.d.d_out, RT));
    reconstruct_kernel<<<grid, 256, 0, st>>>(sign_view(L, 0), sign_view(L, 1), L.UA, L.VA, L.UB, L.VB,
                                             L.d.d_out, L.d.d_in, L.d.k, L.d.l, L.d.env_dtype, W);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

}  // namespace mdbf
