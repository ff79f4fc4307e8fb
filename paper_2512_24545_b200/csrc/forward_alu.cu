// fp32 CUDA-core path of the MDBF forward: any (l, T), any activation type.
//
// One stage computes, for every row r of the sign matrix S (rows x cols):
//
//     out[tau][r] = sum_t U[r][t] * sum_c S[r][c] * ( V[c][t] * in[tau][c] )
//
// i.e. sum_t D_{u_t} S D_{v_t} applied to `in` (Eq. me-dbf-expand): the sign
// matrix is read once per (t, tau) block and shared by the envelope modes; the
// sign is applied by XOR-ing the packed bit into the IEEE sign bit of the
// envelope-scaled activation, so the contraction is add/sub only, accumulated
// in fp32.  Stage B (S_B, V_B, U_B) maps x -> z, stage A (S_A, V_A, U_A) maps
// z -> y.  This is the path of the fp32 configuration and the GPU-side
// cross-check of the tensor-core paths.
#include "common.cuh"

namespace mdbf {

constexpr int ALU_LT = 4;   // envelope modes per pass
constexpr int ALU_TT = 8;   // tokens per pass

template <typename InT, typename OutT>
__global__ void __launch_bounds__(256)
alu_stage_kernel(const SignView words, int rows, int cols,
                 const void *__restrict__ U, const void *__restrict__ V, int l, int env_dtype,
                 const InT *__restrict__ in, OutT *__restrict__ out, int T, int add) {
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (r >= rows) return;
    const int nwords = words.nwords;

    for (int tau0 = 0; tau0 < T; tau0 += ALU_TT) {
        float res[ALU_TT];
#pragma unroll
        for (int b = 0; b < ALU_TT; ++b) res[b] = 0.f;
        for (int t0 = 0; t0 < l; t0 += ALU_LT) {
            float acc[ALU_LT][ALU_TT];
#pragma unroll
            for (int a = 0; a < ALU_LT; ++a)
#pragma unroll
                for (int b = 0; b < ALU_TT; ++b) acc[a][b] = 0.f;
            for (int w = lane; w < nwords; w += 32) {
                const uint32_t word = words.word(r, w);
                const int cmax = min(32, cols - w * 32);
                for (int bit = 0; bit < cmax; ++bit) {
                    const int c = w * 32 + bit;
                    const uint32_t sgn = ((word >> bit) & 1u) << 31;
                    float v[ALU_LT], xv[ALU_TT];
#pragma unroll
                    for (int a = 0; a < ALU_LT; ++a)
                        v[a] = (t0 + a < l) ? env_load(V, (size_t)c * l + t0 + a, env_dtype) : 0.f;
#pragma unroll
                    for (int b = 0; b < ALU_TT; ++b)
                        xv[b] = (tau0 + b < T) ? act_load<InT>(in, (size_t)(tau0 + b) * cols + c) : 0.f;
#pragma unroll
                    for (int a = 0; a < ALU_LT; ++a)
#pragma unroll
                        for (int b = 0; b < ALU_TT; ++b)
                            acc[a][b] += __uint_as_float(__float_as_uint(v[a] * xv[b]) ^ sgn);
                }
            }
            // warp reduction of each accumulator, then the mode contraction with U
#pragma unroll
            for (int a = 0; a < ALU_LT; ++a) {
                const float u = (t0 + a < l) ? env_load(U, (size_t)r * l + t0 + a, env_dtype) : 0.f;
#pragma unroll
                for (int b = 0; b < ALU_TT; ++b) {
                    float s = acc[a][b];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                    res[b] += u * s;
                }
            }
        }
        if (lane == 0) {
#pragma unroll
            for (int b = 0; b < ALU_TT; ++b)
                if (tau0 + b < T) {
                    const size_t o = (size_t)(tau0 + b) * rows + r;
                    act_store<OutT>(out, o, add ? act_load<OutT>(out, o) + res[b] : res[b]);      // add: a further term of a sum
                }
        }
    }
}

template <typename ActT>
static mdbf_status_t run(Layer &L, const void *x, void *y, int T, cudaStream_t st) {
    const int wpb = 8;
    alu_stage_kernel<ActT, float><<<ceil_div(L.d.k, wpb), wpb * 32, 0, st>>>(
        sign_view(L, 1), L.d.k, L.d.d_in, L.UB, L.VB, L.d.l, L.d.env_dtype,
        reinterpret_cast<const ActT *>(x), L.zsum, T, 0);
    MDBF_CUDA(cudaGetLastError());
    if (L.out_mode == 0)
        alu_stage_kernel<float, ActT><<<ceil_div(L.d.d_out, wpb), wpb * 32, 0, st>>>(
            sign_view(L, 0), L.d.d_out, L.d.k, L.UA, L.VA, L.d.l, L.d.env_dtype,
            L.zsum, reinterpret_cast<ActT *>(y), T, 0);
    else                                   // a term of a sum of layers: fp32 output, stored or added
        alu_stage_kernel<float, float><<<ceil_div(L.d.d_out, wpb), wpb * 32, 0, st>>>(
            sign_view(L, 0), L.d.d_out, L.d.k, L.UA, L.VA, L.d.l, L.d.env_dtype,
            L.zsum, reinterpret_cast<float *>(y), T, L.out_mode == 2 ? 1 : 0);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

mdbf_status_t launch_forward_alu(Layer &L, const void *x, void *y, int T, int act_dtype,
                                 cudaStream_t st, int *launches) {
    mdbf_status_t rc;
    if (act_dtype == MDBF_F32) rc = run<float>(L, x, y, T, st);
    else if (act_dtype == MDBF_BF16) rc = run<__nv_bfloat16>(L, x, y, T, st);
    else if (act_dtype == MDBF_F16) rc = run<__half>(L, x, y, T, st);
    else { set_error("mdbf_linear_forward: unsupported activation dtype %d", act_dtype); return MDBF_ERR_DTYPE; }
    if (rc == MDBF_OK) { L.last_ksplit = 0; *launches = 2; }
    return rc;
}

// fp32 accumulator of a sum of layers -> activation type (one rounding)
template <typename OutT>
__global__ void cast_kernel(const float *__restrict__ acc, OutT *__restrict__ y, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        act_store<OutT>(y, i, acc[i]);
}

mdbf_status_t launch_cast(const float *acc, void *y, size_t n, int act_dtype, cudaStream_t st) {
    int grid = (int)((n + 255) / 256);
    if (grid > 148 * 16) grid = 148 * 16;
    if (grid < 1) grid = 1;
    if (act_dtype == MDBF_F32) cast_kernel<float><<<grid, 256, 0, st>>>(acc, reinterpret_cast<float *>(y), n);
    else if (act_dtype == MDBF_BF16) cast_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(acc, reinterpret_cast<__nv_bfloat16 *>(y), n);
    else cast_kernel<__half><<<grid, 256, 0, st>>>(acc, reinterpret_cast<__half *>(y), n);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

// make the fp32 copy of the intermediate current (inspection only): the materialised-envelope kernels keep z in bf16
mdbf_status_t launch_zsum(Layer &L, int T, cudaStream_t st) {
    if (L.last_ksplit < 0) return launch_zb_to_zsum(L, T, st);
    return MDBF_OK;
}

}  // namespace mdbf
