// Internal declarations shared by the libmdbf translation units.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "mdbf.h"

namespace mdbf {

constexpr uint32_t kHandleMagic = 0x4D444246u;  // "MDBF"
constexpr int kMaxL = 64;

// tensor maps of the last materialised-order forward (they depend only on the pointers and T)
struct MatMaps {
    bool valid;
    const void *x, *y;
    int T;
    CUtensorMap tmx, tmz, tmzo, tmyo;
};

// Scratch and pack-time constants of the one-token kernel (forward_t1.cu); index 0 = stage B, 1 = stage A.
struct T1Buffers {
    float *vmax;                  // [2][32] max_c |V[c][t]| per stage and mode
    unsigned int *sync;           // scalars of a forward: max |x|, max |z|
    int8_t *img[2];               // operand images [Np][NB][128]
    int *colsum[2];               // column sums of the images' fixed-point values [Np][32]
    unsigned long long *acc64[2]; // fixed-point sums of the partial outputs of split row blocks [R * 128] (zero between launches)
    int R[2], RG[2], Np[2];       // row blocks, groups of four row blocks, pairs of K blocks
    int NB, ctas;
};

struct Layer {
    mdbf_desc_t d;
    int device;
    // canonical words: kept only by layers without the row-block-major copy below (fp32 envelopes, l > 32)
    uint32_t *wA, *wB;
    int wordsA, wordsB;           // words per row
    // envelopes in env_dtype, row-major [rows][l]
    void *UA, *VA, *UB, *VB;
    // one-token kernels (16-bit envelopes, l <= 32)
    uint16_t *vxA, *vxB;          // bf16 V tile images for the one-token kernel: [kb_pad][max(LP,16)][64], swizzled
    uint2 *wk2A, *wk2B;           // sign words, row-block major [row block][kb_pad][128] (one-token kernel)
    int kbpA, kbpB;               // K blocks per row block in wk2 / vx (even, zero padded)
    // large-T kernel (present only when max_T exceeds the small-T kernel's range and l <= 32):
    int LP;                       // l rounded up to a power of two
    uint2 *wkA, *wkB;             // K-blocked sign words [kblocks][rows_pad128] (tcgen05 kernels)
    int rpA, rpB;                 // rows padded to 128
    int padA, padB;               // reduction length (k, d_in) padded to 64
    float *vtB;                   // V_B transposed, fp32 [LP][padB]
    __nv_bfloat16 *xsB, *xsA;     // pre-scaled operands [xs_rows][padB], [xs_rows][padA]; allocated on first use of the expanded order
    size_t xs_rows;               // max_T * LP rounded up to 256
    CUtensorMap tmB[3], tmA[3];   // tensor maps of xsB / xsA with boxes of 64, 128 and 256 rows (few tokens load a narrow box)
    // materialised-envelope kernel: 16-bit envelope images in mini-MMA operand order (see forward_mat.cu)
    uint16_t *uiA, *uiB;          // U images [row blocks][kcm][16][8][8]
    uint16_t *viA, *viB;          // V images [pairs of K blocks][kcm][16][8][8]
    int kcm;                      // 16-byte chunks of the mode axis: 2 (l <= 16) or 4 (l <= 32)
    __nv_bfloat16 *zb;            // bf16 intermediate [max_T][padA]
    MatMaps mat_maps;
    T1Buffers t1;
    // scratch
    float *zsum;                  // [max_T][k] fp32 intermediate (ALU and one-token kernels; inspection copy otherwise)
    void *xstage, *ystage;        // device staging for the host-buffer entry point
    int32_t *status;              // device status word
    int last_ksplit;              // where the last forward left the intermediate: 0 = zsum, -1 = zb (bf16)
    int out_mode;                 // set per call: 0 y in the activation type; 1 / 2: fp32 y stored / added (a term of a sum)
};

// Bounds-checked build (-DMDBF_BOUNDS_CHECK; `python -m paper_2512_24545_b200.build --bounds-check`): every store of
// a tensor-core forward kernel into the caller's output or into a handle's scratch compares its flat index with the
// extent of the buffer, re-derived from the launch arguments and not from the tile logic that guards the store.  An
// index outside records MDBF_ERR_BOUNDS in the status word and the store is skipped (no trap: the context stays
// usable and the tests read the status).  The normal build compiles the check away.
#ifdef MDBF_BOUNDS_CHECK
__device__ __forceinline__ bool store_in_bounds(size_t idx, size_t extent, int32_t *status) {
    if (idx < extent) return true;
    atomicExch(status, (int32_t)MDBF_ERR_BOUNDS);
    return false;
}
#else
__device__ __forceinline__ bool store_in_bounds(size_t, size_t, int32_t *) { return true; }
#endif

// A packed sign matrix as the kernels that are not tied to one layout read it: the canonical words (layers that only
// the CUDA-core kernels serve), or - tensor-core layers keep a single copy of their signs - the row-block-major
// copy of the one-token kernels, [row block of 128][kb_pad K blocks of 64 columns][128 rows] with 64 bits per entry.
struct SignView {
    const uint32_t *canon;
    const uint2 *wk2;
    int nwords;                   // 32-bit words per row in the canonical layout
    int kb_pad;
    __device__ __forceinline__ uint32_t word(int row, int w) const {
        if (canon) return canon[(size_t)row * nwords + w];
        const uint2 v = wk2[((size_t)(row >> 7) * kb_pad + (w >> 1)) * 128 + (row & 127)];
        return (w & 1) ? v.y : v.x;
    }
};
struct Layer;
SignView sign_view(const Layer &L, int which);      // 0: S_A, 1: S_B

// thread-local error string
void set_error(const char *fmt, ...);
mdbf_status_t cuda_fail(cudaError_t e, const char *what);
// MDBF_OK when the current device is one this library runs on (compute capability 10.x), MDBF_ERR_ARCH otherwise
mdbf_status_t require_device(int *dev_out);
// fp32-accurate dense product on the tensor cores (gemm3x.cu): operand images, then C = A B
size_t gemm3x_image_bytes(int64_t rows, int64_t depth);
mdbf_status_t gemm3x_split(const float *src, size_t stride_i, size_t stride_k, int rows, int depth, uint32_t *img, cudaStream_t st);
mdbf_status_t gemm3x_run(const uint32_t *Aimg, const uint32_t *Bimg, float *C, int n, int r, int depth, int32_t *status, cudaStream_t st,
                         int spare_sms = 0);
// Every device allocation of the library goes through here: cudaMalloc, or - after mdbf_debug_fail_alloc(n) on the
// calling thread - cudaErrorMemoryAllocation for the n-th call from now on without touching the device (the tests
// inject allocation failures this way, on the host).
cudaError_t dev_malloc(void **p, size_t bytes);
template <typename T> inline cudaError_t dev_malloc(T **p, size_t bytes) { return dev_malloc(reinterpret_cast<void **>(p), bytes); }

#define MDBF_CUDA(call)                                                        \
    do {                                                                       \
        cudaError_t e__ = (call);                                              \
        if (e__ != cudaSuccess) return ::mdbf::cuda_fail(e__, #call);          \
    } while (0)

// --- element helpers --------------------------------------------------------
__device__ __forceinline__ float env_load(const void *p, size_t idx, int dtype) {
    if (dtype == MDBF_F16) return __half2float(reinterpret_cast<const __half *>(p)[idx]);
    if (dtype == MDBF_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(p)[idx]);
    return reinterpret_cast<const float *>(p)[idx];
}

template <typename T> __device__ __forceinline__ float act_load(const T *p, size_t i);
template <> __device__ __forceinline__ float act_load<float>(const float *p, size_t i) { return p[i]; }
template <> __device__ __forceinline__ float act_load<__half>(const __half *p, size_t i) { return __half2float(p[i]); }
template <> __device__ __forceinline__ float act_load<__nv_bfloat16>(const __nv_bfloat16 *p, size_t i) { return __bfloat162float(p[i]); }

template <typename T> __device__ __forceinline__ void act_store(T *p, size_t i, float v);
template <> __device__ __forceinline__ void act_store<float>(float *p, size_t i, float v) { p[i] = v; }
template <> __device__ __forceinline__ void act_store<__half>(__half *p, size_t i, float v) { p[i] = __float2half_rn(v); }
template <> __device__ __forceinline__ void act_store<__nv_bfloat16>(__nv_bfloat16 *p, size_t i, float v) { p[i] = __float2bfloat16_rn(v); }

__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// cudaFuncSetAttribute is per device: one flag per (call site, device).  Returns true the first time it is asked
// about the current device (the caller then sets its attributes), false afterwards or when the device is unknown.
struct PerDeviceOnce {
    bool done[64] = {};
    bool first() {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;     // unknown device: set again, it is cheap
        if (done[dev]) return false;
        done[dev] = true;
        return true;
    }
};
inline size_t dtype_size(int dt) { return dt == MDBF_F32 ? 4 : 2; }

// --- launchers (each returns after enqueueing on `st`) ------------------------
mdbf_status_t launch_pack(const int8_t *s, int64_t rows, int64_t cols, uint32_t *out, cudaStream_t st);
mdbf_status_t launch_unpack(const uint32_t *p, int64_t rows, int64_t cols, int8_t *out, cudaStream_t st);
mdbf_status_t launch_env_round(const float *src, void *dst, size_t n, int dtype, cudaStream_t st);
mdbf_status_t launch_env_read(const void *src, float *dst, size_t n, int dtype, cudaStream_t st);
mdbf_status_t launch_kblock(const SignView &sv, int rows, uint2 *out, int rows_pad, int kblocks, cudaStream_t st);
mdbf_status_t launch_canon(const SignView &sv, int rows, uint32_t *out, cudaStream_t st);
mdbf_status_t launch_vtrans(const void *V, int cols, int l, int env_dtype, float *out, int pad, int LP, cudaStream_t st);
mdbf_status_t make_xs_tensor_map(CUtensorMap *out, const void *base, size_t rows, int pad, int box_rows);
mdbf_status_t ensure_prefill_scratch(Layer &L);
mdbf_status_t ensure_kernel_layouts(Layer &L, int kernel, int T);
mdbf_status_t make_act_tensor_map(CUtensorMap *out, const void *base, size_t rows, int cols, int stride, int box_rows);
mdbf_status_t launch_uimg(const void *U, int rows, int l, int env_dtype, uint16_t *out, int rblocks, int kc, cudaStream_t st);
mdbf_status_t launch_forward_mat(Layer &L, const void *x, void *y, int T, cudaStream_t st, int *launches);
bool mat_path_supports(const Layer &L, const void *x, int T);
mdbf_status_t launch_zb_to_zsum(Layer &L, int T, cudaStream_t st);
mdbf_status_t launch_reconstruct(const Layer &L, float *W, cudaStream_t st);
mdbf_status_t launch_forward_alu(Layer &L, const void *x, void *y, int T, int act_dtype,
                                 cudaStream_t st, int *launches);
mdbf_status_t launch_forward_prefill(Layer &L, const void *x, void *y, int T, cudaStream_t st,
                                     int *launches);
mdbf_status_t launch_forward_tmem(Layer &L, const void *x, void *y, int T, cudaStream_t st, int *launches);
bool tmem_path_supports(const Layer &L, int T);
mdbf_status_t launch_forward_tmem_t1(Layer &L, const void *x, void *y, cudaStream_t st);
mdbf_status_t t1_prepare(Layer &L, cudaStream_t st);
void t1_release(Layer &L);
bool t1_supports(const Layer &L);
mdbf_status_t launch_forward_t1_group(Layer *const *Ls, int n, const void *const *xs, void *const *ys, cudaStream_t st, int stages = 3);
constexpr int kMaxSiblings = 4;   // layers one launch of the one-token kernel can serve
int last_t1_launch_count();
mdbf_status_t launch_forward_tmem_t1_sum(Layer *const *Ls, int n, const void *x, float *acc, void *y, cudaStream_t st);
mdbf_status_t launch_forward_tmem_t1_multi(Layer *const *Ls, int n, const void *x, void *const *ys, cudaStream_t st, int stages = 3);
mdbf_status_t launch_wk2(const uint32_t *canon, int rows, int nwords, uint2 *out, int rblocks, int kb_pad,
                         cudaStream_t st);
mdbf_status_t launch_vtile(const void *V, int cols, int l, int env_dtype, uint16_t *out, int kblocks, int NB,
                           cudaStream_t st);
mdbf_status_t launch_wait_timeout_selftest(Layer &L, cudaStream_t st);
mdbf_status_t launch_cast(const float *acc, void *y, size_t n, int act_dtype, cudaStream_t st);
mdbf_status_t launch_zsum(Layer &L, int T, cudaStream_t st);

// host-side canonical packer (pack.cu)
mdbf_status_t host_pack(const int8_t *s, int64_t rows, int64_t cols, uint32_t *out);
mdbf_status_t host_unpack(const uint32_t *p, int64_t rows, int64_t cols, int8_t *out);

}  // namespace mdbf

struct mdbf_handle_s {
    uint32_t magic;
    int32_t kernel;
    int32_t last_launches;
    int32_t last_kernel;
    mdbf::Layer L;
};
