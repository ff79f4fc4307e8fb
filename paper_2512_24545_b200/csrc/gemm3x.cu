// Dense fp32 product C = A B on the tensor cores at close to fp32 accuracy: tcgen05 kind::tf32 and the three-term split
//     a b  ~  a_hi b_hi + a_hi b_lo + a_lo b_hi          (each part a TF32 number; the dropped a_lo b_lo is below 2^-24 a b)
// with fp32 accumulation in tensor memory.  It serves the least-squares step of the ADMM refinement (W V and V^T V,
// Eq. admm-U-tilde), where the FP32 pipe would need five times as long.
//
// Two passes.  split_image_kernel turns an operand into "images": per tile of 128 rows (output rows for A, output
// columns for B) and block of 32 contraction indices one 32 KB piece holding hi (128 rows of 32 TF32 values, 128 bytes
// each) and lo (the same shape behind it), rows K-major with the 128B swizzle a shared-memory matrix descriptor expects
// (16-byte chunk c of row r at position c ^ (r & 7)); tails are zero.  Either operand may be given transposed: an
// element is read at src[i * stride_i + k * stride_k] with one of the strides equal to one.
// gemm3x_kernel: one CTA per SM walks over 128 x 256 tiles of C (two column tiles of B side by side: the stream from L2
// into shared memory, 96 KB per K block, is what bounds the kernel, and a wider tile spends less of it per flop); one
// lane streams the pieces of each K block into a ring by bulk copies, one lane issues  D (+)= A_hi B_hi, D += A_hi B_lo,
// D += A_lo B_hi  (N = 256, four K steps of 8 each), the eight epilogue warps read the accumulators and store.  Every wait is bounded; on expiry the status word is
// set and the tiles still to be written come out as NaN.
#include <algorithm>
#include <cstdint>

#include "common.cuh"
#include "tmem_ptx.cuh"

namespace mdbf {
namespace g3x {

constexpr int TILE = 128, KB = 32;
constexpr int HALF = TILE * KB * 4;            // bytes of the hi (or lo) part of a piece
constexpr int PIECE = 2 * HALF;                // 32 KB
constexpr int STAGES = 2;
constexpr int KCHUNK = 4;                      // K blocks accumulated in tensor memory before the sum moves to fp32 registers
constexpr int STAGE_BYTES = 3 * PIECE;         // A piece, then B_hi of two column tiles, then their B_lo
constexpr int EPI_WARPS = 8;                   // two per quarter of the TMEM lanes, each with half of the tile's columns
constexpr int THREADS = (EPI_WARPS + 2) * 32;  // epilogue warps, loader, issuer
constexpr size_t SMEM = 1024 + (size_t)STAGES * STAGE_BYTES;

// hi = v rounded to the nearest TF32 number (half-ulp add on the bits; the top binade is truncated so that nothing rounds
// up to infinity), lo = the exact residual rounded the same way
__device__ __forceinline__ void split_tf32(float v, uint32_t &hi, uint32_t &lo) {
    const uint32_t b = __float_as_uint(v);
    hi = ((b & 0x7F000000u) == 0x7F000000u ? b : b + 0x1000u) & 0xFFFFE000u;
    lo = (__float_as_uint(v - __uint_as_float(hi)) + 0x1000u) & 0xFFFFE000u;
}
// grid: (K blocks, tiles); block 256 = 128 rows x 2 halves of the 8 chunks
template <bool K_CONTIGUOUS>
__global__ void __launch_bounds__(256) split_image_kernel(const float *__restrict__ src, size_t stride_i, size_t stride_k, int ni, int nk,
                                                          int nkb, uint32_t *__restrict__ img) {
    const int kb = blockIdx.x, it = blockIdx.y;
    unsigned char *piece = reinterpret_cast<unsigned char *>(img) + ((size_t)it * nkb + kb) * PIECE;
    if (K_CONTIGUOUS) {
        // a quarter warp = one row's 128 bytes: whole-line reads, 16-byte writes that cover a row
        const int chunk = threadIdx.x & 7;
        for (int r = threadIdx.x >> 3; r < TILE; r += 32) {
            const int i = it * TILE + r, k0 = kb * KB + 4 * chunk;
            uint32_t h[4], l[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float v = (i < ni && k0 + u < nk) ? src[(size_t)i * stride_i + (size_t)(k0 + u)] : 0.f;
                split_tf32(v, h[u], l[u]);
            }
            const int off = r * 128 + ((chunk ^ (r & 7)) << 4);
            *reinterpret_cast<uint4 *>(piece + off) = make_uint4(h[0], h[1], h[2], h[3]);
            *reinterpret_cast<uint4 *>(piece + HALF + off) = make_uint4(l[0], l[1], l[2], l[3]);
        }
    } else {
        // thread = row (consecutive rows are consecutive in memory), two threads per row share its 8 chunks
        const int r = threadIdx.x & 127, i = it * TILE + r;
        for (int chunk = threadIdx.x >> 7; chunk < 8; chunk += 2) {
            const int k0 = kb * KB + 4 * chunk;
            uint32_t h[4], l[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float v = (i < ni && k0 + u < nk) ? src[(size_t)i + (size_t)(k0 + u) * stride_k] : 0.f;
                split_tf32(v, h[u], l[u]);
            }
            const int off = r * 128 + ((chunk ^ (r & 7)) << 4);
            *reinterpret_cast<uint4 *>(piece + off) = make_uint4(h[0], h[1], h[2], h[3]);
            *reinterpret_cast<uint4 *>(piece + HALF + off) = make_uint4(l[0], l[1], l[2], l[3]);
        }
    }
}

__device__ __forceinline__ void umma_ss_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// instruction descriptor: fp32 accumulator, A and B TF32, both K-major, M = 128
__device__ __forceinline__ uint32_t idesc_tf32(int n) {
    uint32_t d = 0;
    d |= 1u << 4;                       // D: fp32
    d |= 2u << 7;                       // A: tf32
    d |= 2u << 10;                      // B: tf32
    d |= (uint32_t)(n >> 3) << 17;      // N
    d |= (uint32_t)(128 >> 4) << 24;    // M
    return d;
}

// Persistent: CTA c takes the tiles c, c + gridDim.x, ... (row tile = t / ntn2, so that CTAs running side by side share
// their pieces of A in L2).  Two accumulators of 256 tensor-memory columns alternate between tiles: the epilogue of
// one tile runs under the products of the next.  All three terms of a tile accumulate into the same columns, for KCHUNK
// K blocks at a time: the tensor core's accumulation is not rounded to nearest, and its one-sided error grows with the
// number of accumulations (6e-5 of the result over 8192 contraction indices, measured); the chunks' sums are added in
// fp32 by the epilogue, in registers.  ntn is
// the number of 128-column tiles of B's images, ntn2 = ceil(ntn / 2) the number of tiles here; an odd last tile has no
// second half: nothing is copied for it, the products read whatever the buffer holds, and nothing of it is stored.
__global__ void __launch_bounds__(THREADS, 1) gemm3x_kernel(const uint32_t *__restrict__ Aimg, const uint32_t *__restrict__ Bimg,
                                                            float *__restrict__ C, int n, int r, int nkb, int ntn, int ntn2, int ntiles,
                                                            int32_t *__restrict__ status) {
    using namespace tm;
    extern __shared__ unsigned char g3_smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * STAGES + 4];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(g3_smem_raw) + 1023u) & ~1023u;
    const uint32_t full_bar = smem_u32(&bars[0]), empty_bar = smem_u32(&bars[STAGES]);
    const uint32_t acc_full = smem_u32(&bars[2 * STAGES]), acc_empty = smem_u32(&bars[2 * STAGES + 2]);
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar + 8 * s, 1);                      // the loader's expect_tx
            mbar_init(empty_bar + 8 * s, 1);                     // the issuer's commit
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(acc_full + 8 * a, 1);                      // the issuer's commit after a tile's last K block
            mbar_init(acc_empty + 8 * a, EPI_WARPS * 32);        // every epilogue thread, once it has read its part
        }
        abort_flag_s = 0;
        fence_barrier_init();
    }
    if (warp == EPI_WARPS + 1) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512u);             // two accumulators of 256 columns; one CTA per SM
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;

    if (warp < EPI_WARPS) {
        // ===================================== epilogue =====================================
        // thread = one row and one half (128 columns) of the tile; the chunks' sums are added in registers, in fp32
        const int half = warp >> 2;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const bool vec = (r & 3) == 0 && (reinterpret_cast<uintptr_t>(C) & 15u) == 0;
        bool alive = true;
        int it = 0;
        const int nch = nkb > 0 ? (nkb + KCHUNK - 1) / KCHUNK : 1;
        for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
            const int mt = t / ntn2, nt2 = t - mt * ntn2;
            const int row = mt * TILE + (warp & 3) * 32 + lane;
            const int col0 = nt2 * 2 * TILE + half * TILE;
            float sum[TILE];
            for (int ch = 0; ch < nch; ++ch, ++it) {
                const int as = it & 1;
                if (alive) alive = mbar_wait(acc_full + 8 * as, ((uint32_t)(it >> 1)) & 1u, abort_flag, status);
                alive = __all_sync(0xffffffffu, alive);
                tc_fence_after();
                if (alive && nkb > 0) {
#pragma unroll
                    for (int j = 0; j < TILE / 16; ++j) {
                        uint32_t d[16];
                        tmem_ld16(tmem + lane_base + (uint32_t)(as * 2 * TILE + half * TILE + 16 * j), d);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 16; ++e) sum[16 * j + e] = ch == 0 ? __uint_as_float(d[e]) : sum[16 * j + e] + __uint_as_float(d[e]);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < TILE; ++e) sum[e] = alive ? 0.f : __int_as_float(0x7fc00000);
                }
                tc_fence_before();
                if (alive) mbar_arrive(acc_empty + 8 * as);       // the accumulator may be overwritten
            }
            if (row < n && col0 < r) {
                float *out = C + (size_t)row * r + col0;
                if (vec && col0 + TILE <= r) {
#pragma unroll
                    for (int e = 0; e < TILE; e += 4) *reinterpret_cast<float4 *>(out + e) = make_float4(sum[e], sum[e + 1], sum[e + 2], sum[e + 3]);
                } else {
#pragma unroll
                    for (int e = 0; e < TILE; ++e)
                        if (col0 + e < r) out[e] = sum[e];
                }
            }
        }
    } else if (warp == EPI_WARPS) {
        // ====================================== loader ======================================
        if (lane == 0) {
            bool alive = true;
            int g = 0;                                           // K blocks issued so far, over all of this CTA's tiles
            for (int t = blockIdx.x; t < ntiles && alive; t += gridDim.x) {
                const int mt = t / ntn2, nt2 = t - mt * ntn2;
                const bool two = 2 * nt2 + 1 < ntn;              // the tile has a second column tile
                const uint32_t *a_src = Aimg + (size_t)mt * nkb * (PIECE / 4);
                const uint32_t *b0_src = Bimg + (size_t)(2 * nt2) * nkb * (PIECE / 4), *b1_src = b0_src + (size_t)nkb * (PIECE / 4);
                for (int kb = 0; kb < nkb && alive; ++kb, ++g) {
                    const int s = g % STAGES;
                    alive = mbar_wait(empty_bar + 8 * s, (((uint32_t)(g / STAGES)) & 1u) ^ 1u, abort_flag, status);
                    if (!alive) break;
                    const uint32_t dst = smem_base + (uint32_t)(s * STAGE_BYTES);
                    mbar_arrive_expect_tx(full_bar + 8 * s, (uint32_t)(two ? 3 * PIECE : 2 * PIECE));
                    bulk_load(dst, a_src + (size_t)kb * (PIECE / 4), (uint32_t)PIECE, full_bar + 8 * s);
                    const uint32_t *b0 = b0_src + (size_t)kb * (PIECE / 4), *b1 = b1_src + (size_t)kb * (PIECE / 4);
                    bulk_load(dst + (uint32_t)PIECE, b0, (uint32_t)HALF, full_bar + 8 * s);                          // B_hi, first 128 rows
                    bulk_load(dst + (uint32_t)(2 * PIECE), b0 + HALF / 4, (uint32_t)HALF, full_bar + 8 * s);         // B_lo, first 128 rows
                    if (two) {
                        bulk_load(dst + (uint32_t)(PIECE + HALF), b1, (uint32_t)HALF, full_bar + 8 * s);             // B_hi, rows 128..255
                        bulk_load(dst + (uint32_t)(2 * PIECE + HALF), b1 + HALF / 4, (uint32_t)HALF, full_bar + 8 * s);
                    }
                }
            }
        }
        __syncwarp();
    } else {
        // ====================================== issuer ======================================
        if (lane == 0) {
            const uint32_t idesc = idesc_tf32(2 * TILE);
            bool alive = true;
            int g = 0, it = 0;
            const int nch = nkb > 0 ? (nkb + KCHUNK - 1) / KCHUNK : 1;
            for (int t = blockIdx.x; t < ntiles && alive; t += gridDim.x) {
                for (int ch = 0; ch < nch && alive; ++ch, ++it) {
                    const int as = it & 1;
                    alive = mbar_wait(acc_empty + 8 * as, (((uint32_t)(it >> 1)) & 1u) ^ 1u, abort_flag, status);
                    if (!alive) break;
                    tc_fence_after();
                    const uint32_t d = tmem + (uint32_t)(as * 2 * TILE);
                    const int kb_end = min(nkb, (ch + 1) * KCHUNK);
                    for (int kb = ch * KCHUNK; kb < kb_end && alive; ++kb, ++g) {
                        const int s = g % STAGES;
                        alive = mbar_wait(full_bar + 8 * s, ((uint32_t)(g / STAGES)) & 1u, abort_flag, status);
                        if (!alive) break;
                        tc_fence_after();
                        const uint32_t stage = smem_base + (uint32_t)(s * STAGE_BYTES);
                        const uint64_t a_hi = make_smem_desc(stage), a_lo = make_smem_desc(stage + (uint32_t)HALF);
                        const uint64_t b_hi = make_smem_desc(stage + (uint32_t)PIECE), b_lo = make_smem_desc(stage + (uint32_t)(2 * PIECE));
                        const bool fresh = kb == ch * KCHUNK;    // the chunk starts on a cleared accumulator
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)           // 8 TF32 = 32 bytes per K step
                            umma_ss_tf32(d, a_hi + (uint64_t)(2 * ks), b_hi + (uint64_t)(2 * ks), idesc, (!fresh || ks > 0) ? 1u : 0u);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) umma_ss_tf32(d, a_hi + (uint64_t)(2 * ks), b_lo + (uint64_t)(2 * ks), idesc, 1u);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) umma_ss_tf32(d, a_lo + (uint64_t)(2 * ks), b_hi + (uint64_t)(2 * ks), idesc, 1u);
                        umma_commit(empty_bar + 8 * s);
                    }
                    if (alive && nkb > 0) umma_commit(acc_full + 8 * as);
                    else mbar_arrive(acc_full + 8 * as);
                }
            }
        }
        __syncwarp();
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) drain_delay();                              // let copies in flight land before the shared memory goes back
    if (warp == EPI_WARPS + 1) tmem_dealloc(tmem, 512u);
}

}  // namespace g3x

size_t gemm3x_image_bytes(int64_t rows, int64_t depth) {
    return (size_t)ceil_div((int)rows, g3x::TILE) * (size_t)ceil_div((int)depth, g3x::KB) * g3x::PIECE;
}

// images of an operand with `rows` tile rows and `depth` contraction indices; element (i, k) at src[i * stride_i + k * stride_k]
mdbf_status_t gemm3x_split(const float *src, size_t stride_i, size_t stride_k, int rows, int depth, uint32_t *img, cudaStream_t st) {
    const dim3 grid(ceil_div(depth, g3x::KB), ceil_div(rows, g3x::TILE));
    if (stride_k == 1) g3x::split_image_kernel<true><<<grid, 256, 0, st>>>(src, stride_i, stride_k, rows, depth, (int)grid.x, img);
    else if (stride_i == 1) g3x::split_image_kernel<false><<<grid, 256, 0, st>>>(src, stride_i, stride_k, rows, depth, (int)grid.x, img);
    else { set_error("gemm3x_split: one of the strides must be 1"); return MDBF_ERR_INVALID_ARG; }
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

// C (n x r, row-major) = A B from the operands' images (A: n rows, B: r rows, both `depth` deep); spare_sms SMs are left
// to kernels of another stream
mdbf_status_t gemm3x_run(const uint32_t *Aimg, const uint32_t *Bimg, float *C, int n, int r, int depth, int32_t *status, cudaStream_t st,
                         int spare_sms) {
    static PerDeviceOnce once;
    if (once.first()) MDBF_CUDA(cudaFuncSetAttribute(g3x::gemm3x_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g3x::SMEM));
    const int ntm = ceil_div(n, g3x::TILE), ntn = ceil_div(r, g3x::TILE);
    static int sms_of_device[64] = {};
    int dev = 0, sms = 0;
    MDBF_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && sms_of_device[dev]) {
        sms = sms_of_device[dev];
    } else {
        MDBF_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        if (dev >= 0 && dev < 64) sms_of_device[dev] = sms;
    }
    const int ntn2 = ceil_div(ntn, 2), ntiles = ntm * ntn2;
    g3x::gemm3x_kernel<<<std::min(ntiles, std::max(1, sms - spare_sms)), g3x::THREADS, g3x::SMEM, st>>>(Aimg, Bimg, C, n, r, ceil_div(depth, g3x::KB), ntn, ntn2,
                                                                              ntiles, status);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

}  // namespace mdbf
