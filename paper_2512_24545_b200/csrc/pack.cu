// Sign packer / unpacker (canonical layout), kernel-private tiling, envelope rounding.
//
// Canonical layout: 32 signs per uint32 along the row, column c -> word c/32,
// bit c%32 (bit 0 least significant), bit set <=> sign -1, padding bits 0.
#include "common.cuh"

namespace mdbf {

// ------------------------------------------------------------------ host side
mdbf_status_t host_pack(const int8_t *s, int64_t rows, int64_t cols, uint32_t *out) {
    const int64_t nw = (cols + 31) / 32;
    for (int64_t r = 0; r < rows; ++r) {
        const int8_t *row = s + r * cols;
        for (int64_t w = 0; w < nw; ++w) {
            uint32_t word = 0;
            const int64_t c0 = w * 32;
            const int64_t n = (cols - c0 < 32) ? (cols - c0) : 32;
            for (int64_t b = 0; b < n; ++b) {
                const int8_t v = row[c0 + b];
                if (v == -1) word |= (1u << b);
                else if (v != 1) {
                    set_error("mdbf_pack_signs: entry (%lld, %lld) is %d, expected +1 or -1",
                              (long long)r, (long long)(c0 + b), (int)v);
                    return MDBF_ERR_VALUE;
                }
            }
            out[r * nw + w] = word;
        }
    }
    return MDBF_OK;
}

mdbf_status_t host_unpack(const uint32_t *p, int64_t rows, int64_t cols, int8_t *out) {
    const int64_t nw = (cols + 31) / 32;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c)
            out[r * cols + c] = ((p[r * nw + c / 32] >> (c % 32)) & 1u) ? -1 : 1;
    return MDBF_OK;
}

// ---------------------------------------------------------------- device side
// One warp per (row, group of 32 words): lane b of the warp reads column
// 32*w + b (a coalesced 32-byte row segment) and the ballot forms the word.
__global__ void pack_kernel(const int8_t *__restrict__ s, int64_t rows, int64_t cols, int64_t nw,
                            uint32_t *__restrict__ out) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t total = rows * nw;
    for (int64_t item = warp; item < total; item += nwarps) {
        const int64_t r = item / nw, w = item - r * nw;
        const int64_t c = w * 32 + lane;
        const int neg = (c < cols) ? (s[r * cols + c] == -1) : 0;
        const uint32_t word = __ballot_sync(0xffffffffu, neg);
        if (lane == 0) out[item] = word;
    }
}

__global__ void unpack_kernel(const uint32_t *__restrict__ p, int64_t rows, int64_t cols, int64_t nw,
                              int8_t *__restrict__ out) {
    const int64_t total = rows * cols;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = e / cols, c = e - r * cols;
        out[e] = ((p[r * nw + (c >> 5)] >> (c & 31)) & 1u) ? -1 : 1;
    }
}


__global__ void env_round_kernel(const float *__restrict__ src, void *__restrict__ dst, size_t n, int dtype) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float v = src[i];
        if (dtype == MDBF_F16) reinterpret_cast<__half *>(dst)[i] = __float2half_rn(v);
        else if (dtype == MDBF_BF16) reinterpret_cast<__nv_bfloat16 *>(dst)[i] = __float2bfloat16_rn(v);
        else reinterpret_cast<float *>(dst)[i] = v;
    }
}

__global__ void env_read_kernel(const void *__restrict__ src, float *__restrict__ dst, size_t n, int dtype) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = env_load(src, i, dtype);
}

static int grid_for(int64_t items, int per_block) {
    int64_t g = (items + per_block - 1) / per_block;
    if (g < 1) g = 1;
    if (g > 148 * 16) g = 148 * 16;
    return (int)g;
}

mdbf_status_t launch_pack(const int8_t *s, int64_t rows, int64_t cols, uint32_t *out, cudaStream_t st) {
    const int64_t nw = (cols + 31) / 32;
    pack_kernel<<<grid_for(rows * nw, 8), 256, 0, st>>>(s, rows, cols, nw, out);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

mdbf_status_t launch_unpack(const uint32_t *p, int64_t rows, int64_t cols, int8_t *out, cudaStream_t st) {
    const int64_t nw = (cols + 31) / 32;
    unpack_kernel<<<grid_for(rows * cols, 256), 256, 0, st>>>(p, rows, cols, nw, out);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}


mdbf_status_t launch_env_round(const float *src, void *dst, size_t n, int dtype, cudaStream_t st) {
    env_round_kernel<<<grid_for((int64_t)n, 256), 256, 0, st>>>(src, dst, n, dtype);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

mdbf_status_t launch_env_read(const void *src, float *dst, size_t n, int dtype, cudaStream_t st) {
    env_read_kernel<<<grid_for((int64_t)n, 256), 256, 0, st>>>(src, dst, n, dtype);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

}  // namespace mdbf
