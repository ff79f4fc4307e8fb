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
constexpr int kMaxKSplit = 8;          // stage-B partial sums kept per handle
constexpr int kDecodeMaxT = 4;         // tokens per call the small-T kernel takes

// Kernel-private tiled copy of a packed sign matrix (see pack.cu):
// tiles of 32 rows x 128 columns, 512 bytes each, tile (rt, kt) at
// ((rt * ktiles) + kt) * 128 words; inside a tile lane L = 4*g + q of a warp
// owns the uint4 { w(g, q), w(g+8, q), w(g+16, q), w(g+24, q) } where
// w(r, q) is canonical word q of row r of the tile.
struct TiledSigns {
    const uint32_t *words;  // device
    int rtiles;             // ceil(rows / 32)
    int ktiles;             // ceil(cols / 128)
};

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
    unsigned int *sync;           // scalars of a forward: column sums of the fixed-point operand, max |x|, max |z|
    int8_t *img[2];               // operand images [Np][NB][128]
    unsigned long long *acc64[2]; // fixed-point sums of the partial outputs of split row blocks [R * 128] (zero between launches)
    int R[2], RG[2], Np[2];       // row blocks, groups of four row blocks, pairs of K blocks
    int NB, ctas;
};

struct Layer {
    mdbf_desc_t d;
    int device;
    // canonical words
    uint32_t *wA, *wB;
    int wordsA, wordsB;           // words per row
    // tiled words
    uint32_t *tA, *tB;
    int rtA, ktA, rtB, ktB;
    // envelopes in env_dtype, row-major [rows][l]
    void *UA, *VA, *UB, *VB;
    // kernel-private bf16 copies of V_A / V_B in MMA B-fragment order (see forward_decode.cu)
    uint2 *vfA, *vfB;
    int NT;                       // 8-column mode tiles in the fragment copies: 1, 2, 4 or 8
    // TMEM-operand small-T kernel (16-bit envelopes, l <= 32): V in MMA k order, 16-bit, [kblocks][LP][64]
    uint16_t *vpA, *vpB;
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
    float *z;                     // [kMaxKSplit][zT][k] stage-B partial sums of the small-T kernel
    size_t zstride;               // zT * k
    float *zsum;                  // [max_T][k] summed intermediate (ALU path, inspection)
    void *xstage, *ystage;        // device staging for the host-buffer entry point
    int32_t *status;              // device status word
    int last_ksplit;              // how many partials the last forward wrote (0 = zsum valid, -1 = the intermediate is in zb)
    int out_mode;                 // set per call: 0 y in the activation type; 1 / 2: fp32 y stored / added (a term of a sum)
};

// thread-local error string
void set_error(const char *fmt, ...);
mdbf_status_t cuda_fail(cudaError_t e, const char *what);

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
inline size_t dtype_size(int dt) { return dt == MDBF_F32 ? 4 : 2; }

// --- launchers (each returns after enqueueing on `st`) ------------------------
mdbf_status_t launch_pack(const int8_t *s, int64_t rows, int64_t cols, uint32_t *out, cudaStream_t st);
mdbf_status_t launch_unpack(const uint32_t *p, int64_t rows, int64_t cols, int8_t *out, cudaStream_t st);
mdbf_status_t launch_tile(const uint32_t *canon, int rows, int words, uint32_t *tiled, int rtiles,
                          int ktiles, cudaStream_t st);
mdbf_status_t launch_env_round(const float *src, void *dst, size_t n, int dtype, cudaStream_t st);
mdbf_status_t launch_env_read(const void *src, float *dst, size_t n, int dtype, cudaStream_t st);
mdbf_status_t launch_vfrag(const void *V, int cols, int l, int env_dtype, uint2 *out, int ktiles, int NT,
                           cudaStream_t st);
mdbf_status_t launch_kblock(const uint32_t *canon, int rows, int nwords, uint2 *out, int rows_pad, int kblocks,
                            cudaStream_t st);
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
mdbf_status_t launch_forward_decode(Layer &L, const void *x, void *y, int T, cudaStream_t st,
                                    int *launches);
mdbf_status_t launch_forward_prefill(Layer &L, const void *x, void *y, int T, cudaStream_t st,
                                     int *launches);
mdbf_status_t launch_forward_tmem(Layer &L, const void *x, void *y, int T, cudaStream_t st, int *launches);
bool tmem_path_supports(const Layer &L, int T);
mdbf_status_t launch_vperm(const void *V, int cols, int l, int env_dtype, uint16_t *out, int kblocks, int LP,
                           cudaStream_t st);
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
