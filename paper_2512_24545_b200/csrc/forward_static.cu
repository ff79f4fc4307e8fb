// mdbf_linear_forward_static: the fp32 CUDA-core forward for callers that cannot allocate.
//
// Who needs it: code that runs after its process has handed all device memory to an arena of
// its own (a serving runtime that forbids cudaMalloc once it is up, a plug-in that only
// receives buffers from its host application, a real-time loop where an allocation's implicit
// device synchronisation is not acceptable).  Such a caller cannot build a layer handle,
// because mdbf_pack allocates; it lays the canonical packed words and the envelope factors out
// in buffers it already owns and passes them here together with x and y.
//
// The one piece of memory the computation needs beyond its inputs and outputs is the k x T
// intermediate z between the two stages.  Here it lives in a file-scope device array of fixed
// size that every GPU loading the library carries until the process exits, so the entry point
// calls no cudaMalloc, no cudaFree and no allocating library routine.
//
// The arithmetic is that of the handle-based fp32 path (forward_alu.cu): per stage
// out[tau][r] = sum_t U[r][t] * sum_c S[r][c] * (V[c][t] * in[tau][c]), the sign applied by
// XOR-ing the packed bit into the IEEE sign bit, fp32 accumulation, lanes striding over the
// packed words of a row and a butterfly reduction at the end.
#include <mutex>

#include "common.cuh"

namespace mdbf {

// Capacity of the shared intermediate, in floats (1 MiB).  A call needs k * T of them.
constexpr size_t kStaticZFloats = MDBF_STATIC_MAX_KT;

// In host code this name is only a stand-in for the symbol; the device address is obtained
// once per device with cudaGetSymbolAddress (static_z_address below).
static __device__ __align__(256) float g_static_z[kStaticZFloats];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mutex;
static float *g_static_z_ptr[kMaxDevices] = {};

// Device address of g_static_z on the current device; first call per device does the set-up.
static mdbf_status_t static_z_address(float **out) {
    int n = 0;
    cudaError_t e = cudaGetDeviceCount(&n);
    if (e != cudaSuccess || n == 0) {
        cudaGetLastError();
        set_error("mdbf_linear_forward_static needs a CUDA device of compute capability 10.x; none is visible");
        return MDBF_ERR_ARCH;
    }
    int dev = 0;
    MDBF_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) {
        set_error("mdbf_linear_forward_static: device ordinal %d is outside [0, %d)", dev, kMaxDevices);
        return MDBF_ERR_INVALID_ARG;
    }
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_z_ptr[dev]) {
        int major = 0;
        MDBF_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
        if (major != 10) {
            set_error("libmdbf is built for sm_100a only; device %d has compute capability major %d", dev, major);
            return MDBF_ERR_ARCH;
        }
        float *p = nullptr;
        MDBF_CUDA(cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_static_z));
        if (!p) {
            set_error("mdbf_linear_forward_static: cudaGetSymbolAddress returned a null address");
            return MDBF_ERR_CUDA;
        }
        g_static_z_ptr[dev] = p;
    }
    *out = g_static_z_ptr[dev];
    return MDBF_OK;
}

constexpr int ST_LT = 4;   // envelope modes per pass
constexpr int ST_TT = 8;   // tokens per pass

// One warp per row of the sign matrix; writes every out[tau][r] it owns (nothing accumulates
// into `out`, so the shared intermediate needs no clearing between calls).
template <typename InT, typename OutT>
__global__ void __launch_bounds__(256)
static_stage_kernel(const uint32_t *__restrict__ words, int nwords, int rows, int cols,
                    const void *__restrict__ U, const void *__restrict__ V, int l, int env_dtype,
                    const InT *__restrict__ in, OutT *__restrict__ out, int T) {
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (r >= rows) return;
    const uint32_t *wrow = words + (size_t)r * nwords;
    for (int tau0 = 0; tau0 < T; tau0 += ST_TT) {
        float res[ST_TT];
#pragma unroll
        for (int b = 0; b < ST_TT; ++b) res[b] = 0.f;
        for (int t0 = 0; t0 < l; t0 += ST_LT) {
            float acc[ST_LT][ST_TT];
#pragma unroll
            for (int a = 0; a < ST_LT; ++a)
#pragma unroll
                for (int b = 0; b < ST_TT; ++b) acc[a][b] = 0.f;
            for (int w = lane; w < nwords; w += 32) {
                const uint32_t word = wrow[w];
                const int cmax = min(32, cols - w * 32);
                for (int bit = 0; bit < cmax; ++bit) {
                    const int c = w * 32 + bit;
                    const uint32_t sgn = ((word >> bit) & 1u) << 31;
                    float v[ST_LT], xv[ST_TT];
#pragma unroll
                    for (int a = 0; a < ST_LT; ++a)
                        v[a] = (t0 + a < l) ? env_load(V, (size_t)c * l + t0 + a, env_dtype) : 0.f;
#pragma unroll
                    for (int b = 0; b < ST_TT; ++b)
                        xv[b] = (tau0 + b < T) ? act_load<InT>(in, (size_t)(tau0 + b) * cols + c) : 0.f;
#pragma unroll
                    for (int a = 0; a < ST_LT; ++a)
#pragma unroll
                        for (int b = 0; b < ST_TT; ++b)
                            acc[a][b] += __uint_as_float(__float_as_uint(v[a] * xv[b]) ^ sgn);
                }
            }
#pragma unroll
            for (int a = 0; a < ST_LT; ++a) {
                const float u = (t0 + a < l) ? env_load(U, (size_t)r * l + t0 + a, env_dtype) : 0.f;
#pragma unroll
                for (int b = 0; b < ST_TT; ++b) {
                    float s = acc[a][b];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                    res[b] += u * s;
                }
            }
        }
        if (lane == 0) {
#pragma unroll
            for (int b = 0; b < ST_TT; ++b)
                if (tau0 + b < T) act_store<OutT>(out, (size_t)(tau0 + b) * rows + r, res[b]);
        }
    }
}

template <typename ActT>
static mdbf_status_t run_static(const mdbf_desc_t &d, const uint32_t *wA, const uint32_t *wB, const void *UA,
                                const void *VA, const void *UB, const void *VB, const void *x, void *y, int T,
                                float *z, cudaStream_t st) {
    const int wpb = 8;
    static_stage_kernel<ActT, float><<<ceil_div(d.k, wpb), wpb * 32, 0, st>>>(
        wB, ceil_div(d.d_in, 32), d.k, d.d_in, UB, VB, d.l, d.env_dtype, reinterpret_cast<const ActT *>(x), z, T);
    MDBF_CUDA(cudaGetLastError());
    static_stage_kernel<float, ActT><<<ceil_div(d.d_out, wpb), wpb * 32, 0, st>>>(
        wA, ceil_div(d.k, 32), d.d_out, d.k, UA, VA, d.l, d.env_dtype, z, reinterpret_cast<ActT *>(y), T);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

}  // namespace mdbf

using namespace mdbf;

extern "C" mdbf_status_t mdbf_linear_forward_static(const mdbf_desc_t *desc, const uint32_t *wA, const uint32_t *wB,
                                                    const void *U_A, const void *V_A, const void *U_B,
                                                    const void *V_B, const void *x, void *y, int32_t T,
                                                    int32_t act_dtype, void *stream) {
    if (!desc || !wA || !wB || !U_A || !V_A || !U_B || !V_B || !x || !y) {
        set_error("mdbf_linear_forward_static: NULL pointer");
        return MDBF_ERR_INVALID_ARG;
    }
    const mdbf_desc_t d = *desc;
    if (d.d_out < 1 || d.d_in < 1 || d.k < 1 || d.l < 1 || d.l > kMaxL || T < 1) {
        set_error("mdbf_linear_forward_static: bad shape d_out=%d d_in=%d k=%d l=%d T=%d (need all >= 1, l <= %d)",
                  d.d_out, d.d_in, d.k, d.l, T, kMaxL);
        return MDBF_ERR_SHAPE;
    }
    if ((size_t)d.k * (size_t)T > kStaticZFloats) {
        set_error("mdbf_linear_forward_static: k * T = %zu exceeds the built-in scratch of %zu floats "
                  "(MDBF_STATIC_MAX_KT); use mdbf_pack + mdbf_linear_forward for larger calls",
                  (size_t)d.k * (size_t)T, kStaticZFloats);
        return MDBF_ERR_SHAPE;
    }
    const bool env_ok = d.env_dtype == MDBF_F32 || d.env_dtype == MDBF_F16 || d.env_dtype == MDBF_BF16;
    const bool act_ok = act_dtype == MDBF_F32 || act_dtype == MDBF_F16 || act_dtype == MDBF_BF16;
    if (!env_ok || !act_ok) {
        set_error("mdbf_linear_forward_static: unsupported dtype (env %d, act %d)", d.env_dtype, act_dtype);
        return MDBF_ERR_DTYPE;
    }
    float *z = nullptr;
    mdbf_status_t rc = static_z_address(&z);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (act_dtype == MDBF_F32) return run_static<float>(d, wA, wB, U_A, V_A, U_B, V_B, x, y, T, z, st);
    if (act_dtype == MDBF_BF16) return run_static<__nv_bfloat16>(d, wA, wB, U_A, V_A, U_B, V_B, x, y, T, z, st);
    return run_static<__half>(d, wA, wB, U_A, V_A, U_B, V_B, x, y, T, z, st);
}
