// Multi-Envelope SVID on the GPU:  MSVID_l[Z] = sign(Z) (.) TSVD_l(|Z|)   (Eq. msvid-def), the operator the paper
// applies to the balanced factors of a weight matrix to initialise MDBF (Eq. mesvid-init-compact) and, by
// Theorem 1 (Eq. rankl-error / Eq. Ustar), the best approximation of Z among all matrices that keep Z's sign mask
// and have an envelope of rank <= l.
//
// The sign mask is exact (bit set <=> entry negative, sign(0) = +1: the Notation section), written in the
// library's canonical packing.  The truncated SVD of the demodulated envelope |Z| (N x M, never stored: every pass
// takes the absolute value on the fly) is computed by block subspace iteration on a block of l columns:
//
//     Q  <- orth(Q0)                                 M x l start block, passed in by the caller
//     repeat n_iter times:   Y <- orth(|Z| Q);   Q <- orth(|Z|^T Y)
//     Y  <- |Z| Q;   Y^T Y = W diag(s^2) W^T        (l x l symmetric eigenproblem, Jacobi)
//     U  <- Y W diag(s^-1/2),   V <- Q W diag(s^1/2)      balanced factors:  U V^T = Y Q^T ~ TSVD_l(|Z|)
//
// Two passes over Z per iteration, each a tall-skinny product.  At l = 16 that is 16 FMAs per 4 bytes of Z: on the
// CUDA cores the FP32 pipe needs as long as HBM does, so the products run on the tensor cores
// (envelope_product_tc_kernel: TF32 operands in a three-term split, the envelope written straight into tensor
// memory) and reach three quarters of the memory rate; the scalar kernels absz_q_kernel / abszT_y_kernel serve the
// shapes a tensor map cannot take.  The first pass also packs the sign mask.  orth() is a Cholesky QR with the
// l x l Gram matrix accumulated and factorised in fp64, one launch for the Gram matrix, its reduction and its factor.  What the iteration
// leaves short of the exact TSVD is the mixing among the nearly equal singular values of the bulk: the largest
// singular value converges in two iterations, the squared error of the envelope stays within a fraction of a
// per cent of the optimum of Theorem 1 (the GPU tests bound it), and every Ritz value is a lower bound of the
// singular value it estimates.
#include <algorithm>
#include <cmath>

#include "common.cuh"
#include "tmem_ptx.cuh"

namespace mdbf {
namespace msv {

constexpr int kMaxL = 32;

// ------------------------------------------------------------------ sign mask
// Bit c % 32 of word c / 32 is set <=> Z[r][c] is negative (a NaN counts as negative, as in the comparison
// `not (z >= 0)` that defines sign() with sign(0) = +1); padding bits are 0.  CTA = one row x 2048 columns, a warp
// takes eight words: eight independent 128-byte loads per lane, one ballot per word.
constexpr int SP_WORDS = 8;
__global__ void __launch_bounds__(256) sign_pack_kernel(const float *__restrict__ Z, int q, int nwords, uint32_t *__restrict__ out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t r = blockIdx.x;
    const int w0 = (blockIdx.y * 8 + warp) * SP_WORDS;
    const float *zr = Z + r * (size_t)q;
    float z[SP_WORDS];
#pragma unroll
    for (int u = 0; u < SP_WORDS; ++u) {
        const int c = (w0 + u) * 32 + lane;
        z[u] = c < q ? zr[c] : 0.f;
    }
    uint32_t mine = 0u;
#pragma unroll
    for (int u = 0; u < SP_WORDS; ++u) {
        const uint32_t bits = __ballot_sync(0xffffffffu, !(z[u] >= 0.f));
        if (lane == u) mine = bits;
    }
    if (lane < SP_WORDS && w0 + lane < nwords) out[r * nwords + w0 + lane] = mine;
}

// ------------------------------------------------------------------ Y = |Z| Q
// CTA = 8 warps x 2 rows.  A lane owns the columns lane, lane + 32, ... of a tile of 256 columns and keeps 2 x LP
// partial sums in registers; the tile's rows of Q (M x LP, zero beyond the l real columns) sit in shared memory,
// [column][LP + 4] (the padding keeps the 128-bit reads of consecutive lanes on different banks), and serve both rows.
// The next tile is in flight while the current one is consumed: its entries of Z are loaded into registers and its
// rows of Q copied asynchronously into the other half of a double buffer (one barrier per tile).  Among 4, 8 or 16
// warps x 1, 2 or 4 rows and tiles of 128 to 512 columns this shape timed best; without the prefetch it is 25 %
// slower.  MASKED: the envelope is S (.) Z for a given packed mask S (bit set <=> -1) instead of |Z| = sign(Z) (.) Z.
constexpr int AQ_WARPS = 8, AQ_ROWS = 2, AQ_TJ = 256;
__device__ __forceinline__ void cp_async16(void *smem, const void *gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
template <int LP, bool MASKED>
__global__ void __launch_bounds__(AQ_WARPS * 32) absz_q_kernel(const float *__restrict__ Z, int p, int q, const float *__restrict__ Q,
                                                              float *__restrict__ Y, const uint32_t *__restrict__ S, int nwords) {
    constexpr int TJ = LP > 16 ? 128 : AQ_TJ, STEPS = TJ / 32;    // l > 16: half the tile, so that the double buffer fits 48 KB
    constexpr int QST = LP + 4;
    constexpr bool ASYNC = LP % 4 == 0;                          // rows of Q are whole 16-byte chunks
    __shared__ __align__(16) float Qs[2][TJ * QST];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = (blockIdx.x * AQ_WARPS + warp) * AQ_ROWS;
    float acc[AQ_ROWS][LP];
#pragma unroll
    for (int r = 0; r < AQ_ROWS; ++r)
#pragma unroll
        for (int t = 0; t < LP; ++t) acc[r][t] = 0.f;
    auto load_q = [&](int j0, int buf) {                         // rows j0 .. j0 + 255 of Q into half `buf`
        if (ASYNC) {
            for (int e = threadIdx.x; e < TJ * (LP / 4 > 0 ? LP / 4 : 1); e += AQ_WARPS * 32) {
                const int jj = e / (LP / 4 > 0 ? LP / 4 : 1), t4 = e - jj * (LP / 4 > 0 ? LP / 4 : 1);
                float *dst = &Qs[buf][jj * QST + 4 * t4];
                if (j0 + jj < q) cp_async16(dst, Q + (size_t)(j0 + jj) * LP + 4 * t4);
                else *reinterpret_cast<float4 *>(dst) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        } else {
            for (int e = threadIdx.x; e < TJ * LP; e += AQ_WARPS * 32) {
                const int jj = e / LP, t = e - jj * LP;
                Qs[buf][jj * QST + t] = j0 + jj < q ? Q[(size_t)(j0 + jj) * LP + t] : 0.f;
            }
        }
        asm volatile("cp.async.commit_group;\n" ::: "memory");
    };
    auto load_z = [&](int j0, float (&z)[AQ_ROWS][STEPS]) {
#pragma unroll
        for (int r = 0; r < AQ_ROWS; ++r)
#pragma unroll
            for (int s = 0; s < STEPS; ++s) {
                const int j = j0 + s * 32 + lane;
                float v = (r0 + r < p && j < q) ? Z[(size_t)(r0 + r) * q + j] : 0.f;
                if (MASKED) {
                    const uint32_t w = (r0 + r < p && j0 + s * 32 < q) ? S[(size_t)(r0 + r) * nwords + ((j0 >> 5) + s)] : 0u;   // one word per warp
                    v = __uint_as_float(__float_as_uint(v) ^ (((w >> lane) & 1u) << 31));
                } else {
                    v = fabsf(v);
                }
                z[r][s] = v;
            }
    };
    float zc[AQ_ROWS][STEPS], zn[AQ_ROWS][STEPS];
    load_z(0, zc);
    load_q(0, 0);
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
    __syncthreads();
    int buf = 0;
    for (int j0 = 0; j0 < q; j0 += TJ, buf ^= 1) {
        const bool more = j0 + TJ < q;
        if (more) {
            load_q(j0 + TJ, buf ^ 1);
            load_z(j0 + TJ, zn);
        }
#pragma unroll
        for (int s = 0; s < STEPS; ++s) {
            const float *qrow = &Qs[buf][(s * 32 + lane) * QST];
            if (ASYNC) {
#pragma unroll
                for (int t4 = 0; t4 < LP / 4; ++t4) {
                    const float4 qv = *reinterpret_cast<const float4 *>(qrow + 4 * t4);
#pragma unroll
                    for (int r = 0; r < AQ_ROWS; ++r) {
                        acc[r][4 * t4] = fmaf(zc[r][s], qv.x, acc[r][4 * t4]);
                        acc[r][4 * t4 + 1] = fmaf(zc[r][s], qv.y, acc[r][4 * t4 + 1]);
                        acc[r][4 * t4 + 2] = fmaf(zc[r][s], qv.z, acc[r][4 * t4 + 2]);
                        acc[r][4 * t4 + 3] = fmaf(zc[r][s], qv.w, acc[r][4 * t4 + 3]);
                    }
                }
            } else {
#pragma unroll
                for (int t = 0; t < LP; ++t) {
                    const float qv = qrow[t];
#pragma unroll
                    for (int r = 0; r < AQ_ROWS; ++r) acc[r][t] = fmaf(zc[r][s], qv, acc[r][t]);
                }
            }
        }
        asm volatile("cp.async.wait_group 0;\n" ::: "memory");
        __syncthreads();                                         // the other half is complete, this half is free
        if (more) {
#pragma unroll
            for (int r = 0; r < AQ_ROWS; ++r)
#pragma unroll
                for (int s = 0; s < STEPS; ++s) zc[r][s] = zn[r][s];
        }
    }
#pragma unroll
    for (int r = 0; r < AQ_ROWS; ++r)
#pragma unroll
        for (int t = 0; t < LP; ++t) {
            float v = acc[r][t];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0 && r0 + r < p) Y[(size_t)(r0 + r) * LP + t] = v;
        }
}

// ------------------------------------------------------------------ Y = |Z| Q and W = |Z|^T Y on the tensor cores
// The two products of the subspace iteration with tcgen05 (kind::tf32, fp32 accumulators in tensor memory) and a
// three-term split of the fp32 operands:  e = e_hi + e_lo,  q = q_hi + q_lo  (each part a TF32 number),
//     e q  ~  e_hi q_hi + e_hi q_lo + e_lo q_hi                      (the dropped e_lo q_lo is below 2^-24 e q).
// CTA = 128 output rows x a range of K blocks of 32 (split over blockIdx.y, partial sums per range).  Per K block:
//   one lane brings the raw 128 x 32 tile of Z into a ring of buffers by TMA (zero fill outside the matrix), so the
//     bytes in flight do not depend on how many threads wait for them;
//   8 converter warps (two groups on alternate K blocks, thread = output row = TMEM lane) read their row of the tile,
//     take the envelope (absolute value, or the sign flipped by the given mask), split it and store E_hi and E_lo
//     straight into tensor memory as the A operand: shared memory carries each byte of Z once in and once out,
//     where operand tiles in shared memory would carry it six times and bound the kernel;
//   one lane bulk-copies the K block's image of the other factor: rows [0, LPP) = q_hi, [LPP, 2 LPP) = q_lo of the 32
//     contraction indices, already in the K-major 128B-swizzled operand layout (right_mul_kernel writes the images
//     when it writes the factor);
//   two lanes issue the MMAs, four K steps of 8 each: D1 (+)= E_hi [q_hi | q_lo] (N = 2 LPP), D2 (+)= E_lo q_hi (N = LPP).
// Epilogue: y[t] = D1[t] + D1[LPP + t] + D2[t] into the range's partial sums.
// TRANS = false: Y = E Q    (output rows = rows of Z, contraction over its columns; TMA box of 32 columns x 128 rows,
//                            128B-swizzled so that a thread's 16-byte reads of its own row spread over the banks)
// TRANS = true:  W = E^T Y  (output rows = columns of Z, contraction over its rows; box of 128 columns x 32 rows)
// Needs cols % 4 == 0 and Z on a 16-byte boundary (the tensor map's rules); other inputs take the scalar kernels.
// Every wait is bounded; on expiry the status word of the workspace is set and the call's outputs are NaN.
constexpr int TC_KB = 32, TC_CONVERTERS = 256;
constexpr int TC_W_ISSUE = 8, TC_W_RAW = 10, TC_W_IMG = 11, TC_THREADS = 12 * 32;
constexpr int TC_TILE = 128 * TC_KB * 4;                        // bytes of a raw tile
constexpr int TC_RAW = 5;                                       // raw tiles in flight per CTA
template <int LP> struct TcCfg {
    static constexpr int LPP = LP < 16 ? 16 : LP;              // MMA N is a multiple of 16
    static constexpr int N1 = 2 * LPP, N2 = LPP;
    static constexpr int IMG = N1 * 128;                        // bytes of one K block's image of the other factor
    static constexpr int ACC_COLS = N1 + N2 <= 64 ? 64 : 128;   // tensor memory: accumulators, then the A stages of 64 columns
    static constexpr int STAGES = (256 - ACC_COLS) / 64;        // two CTAs share the SM's 512 columns
    static constexpr int TMEM_COLS = 256;
    static constexpr size_t SMEM = 1024 + (size_t)TC_RAW * TC_TILE + (size_t)STAGES * IMG;
};
__device__ __forceinline__ uint32_t tf32_round(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;\n" : "=r"(r) : "f"(x));
    return r;
}
// e = hi + lo with hi = e rounded to the nearest TF32 number (an integer half-ulp add on the bits, then the low 13 bits
// cleared; values in the top binade are truncated instead so that nothing rounds up to infinity), the residual e - hi
// exact in fp32, and lo that residual rounded the same way: plain ALU work (the cvt instruction runs on the quarter-rate
// pipe).  |e - hi - lo| <= 2^-24 |e|.
__device__ __forceinline__ void tf32_split(float e, uint32_t &hi, uint32_t &lo) {
    const uint32_t b = __float_as_uint(e);
    hi = ((b & 0x7F000000u) == 0x7F000000u ? b : b + 0x1000u) & 0xFFFFE000u;
    lo = (__float_as_uint(e - __uint_as_float(hi)) + 0x1000u) & 0xFFFFE000u;
}
// D[tmem] (+)= A[tmem] * B[smem], TF32 operands
__device__ __forceinline__ void umma_ts_tf32(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// instruction descriptor: fp32 accumulator, A and B TF32, both K-major, M = 128
__device__ __forceinline__ uint32_t make_idesc_tf32(int n) {
    uint32_t d = 0;
    d |= 1u << 4;                       // D: fp32
    d |= 2u << 7;                       // A: tf32
    d |= 2u << 10;                      // B: tf32
    d |= (uint32_t)(n >> 3) << 17;      // N
    d |= (uint32_t)(128 >> 4) << 24;    // M
    return d;
}
// WRITE_MASK (plain product of |Z| only): the converters also pack the signs of what they read into S_out, the mask of
// Eq. msvid-def (bit = 1 where the entry is below zero; zeros of either sign count as +1), so that the first pass over Z
// yields it for free.
template <int LP, bool MASKED, bool TRANS, bool WRITE_MASK>
__global__ void __launch_bounds__(TC_THREADS, 2) envelope_product_tc_kernel(const __grid_constant__ CUtensorMap tmap_z, int p, int q,
                                                                  const uint32_t *__restrict__ img, int kb_per_cta, float *__restrict__ P,
                                                                  const uint32_t *__restrict__ S, uint32_t *__restrict__ S_out, int nwords,
                                                                  int32_t *__restrict__ status) {
    static_assert(!WRITE_MASK || (!MASKED && !TRANS), "the mask is written by the plain product of |Z|");
    using namespace tm;
    using C = TcCfg<LP>;
    constexpr int LPP = C::LPP, N1 = C::N1, N2 = C::N2, TC_STAGES = C::STAGES;
    extern __shared__ unsigned char tc_smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * TC_STAGES + 2 * TC_RAW + 1];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(tc_smem_raw) + 1023u) & ~1023u;
    unsigned char *smem_gen = tc_smem_raw + (smem_base - smem_u32(tc_smem_raw));
    const uint32_t img_base = smem_base + (uint32_t)(TC_RAW * TC_TILE);
    const uint32_t full_bar = smem_u32(&bars[0]), empty_bar = smem_u32(&bars[TC_STAGES]);
    const uint32_t raw_full = smem_u32(&bars[2 * TC_STAGES]), raw_empty = smem_u32(&bars[2 * TC_STAGES + TC_RAW]);
    const uint32_t accum_bar = smem_u32(&bars[2 * TC_STAGES + 2 * TC_RAW]);
    const int m_ext = TRANS ? q : p, k_ext = TRANS ? p : q;
    // Order of the CTAs over Z, so that a pass starts on what the pass before it read last and finds part of it in L2:
    // W = E^T Y walks the row ranges from the top down (x = column block fastest, y = row range); Y = E Q then walks the
    // row blocks from the bottom up, all column ranges of a row block together.
    int bx = blockIdx.x, by = blockIdx.y;
    if (!TRANS) {
        const int lin = blockIdx.x + gridDim.x * blockIdx.y;
        by = lin % gridDim.y;
        bx = gridDim.x - 1 - lin / gridDim.y;
    }
    const int row0 = bx * 128;                                   // first output row (a row of Z, or a column when TRANS)
    const int nkb_total = (k_ext + TC_KB - 1) / TC_KB;
    const int kb0 = by * kb_per_cta;
    const int nkb = max(0, min(kb_per_cta, nkb_total - kb0));
    if (tid == 0) {
        for (int s = 0; s < TC_STAGES; ++s) {
            mbar_init(full_bar + 8 * s, 4 + 1);                  // the four warps of a converter group + the image's expect_tx
            mbar_init(empty_bar + 8 * s, 2);                     // the two issuing lanes (commits)
        }
        for (int s = 0; s < TC_RAW; ++s) {
            mbar_init(raw_full + 8 * s, 1);                      // the tile's expect_tx
            mbar_init(raw_empty + 8 * s, 4);                     // the four warps of the group that read it
        }
        mbar_init(accum_bar, 2);
        abort_flag_s = 0;
        fence_barrier_init();
    }
    if (warp == TC_W_ISSUE) {
        tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)C::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    const uint32_t tmem_a0 = tmem + (uint32_t)C::ACC_COLS;       // A stage s: columns [64 s, 64 s + 32) = E_hi, the next 32 = E_lo

    if (warp < TC_CONVERTERS / 32) {
        // ============================ converters, then epilogue ============================
        const int grp = warp >> 2;                               // K blocks grp, grp + 2, ...
        const int r = (warp & 3) * 32 + lane;                    // output row within the tile = TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const int wcol = (row0 >> 5) + (warp & 3);               // TRANS: the warp's 32 columns are one packed word per row of Z
        // mask word(s) of K block kb: a thread's own row and the block's word (plain), or lane i = the block's row i (TRANS)
        auto mask_word = [&](int kb) -> uint32_t {
            if (!MASKED || kb >= nkb) return 0u;
            if (TRANS) {
                const int gr = (kb0 + kb) * TC_KB + lane;
                return (gr < p && wcol < nwords) ? S[(size_t)gr * nwords + wcol] : 0u;
            }
            return row0 + r < p ? S[(size_t)(row0 + r) * nwords + kb0 + kb] : 0u;
        };
        bool alive = true;
        uint32_t word = mask_word(grp);
        for (int kb = grp; kb < nkb && alive; kb += 2) {
            const int s = kb % TC_STAGES, rs = kb % TC_RAW;
            const uint32_t word_next = mask_word(kb + 2);        // travels while this block is converted
            alive = mbar_wait(raw_full + 8 * rs, ((uint32_t)(kb / TC_RAW)) & 1u, abort_flag, status);
            if (alive) alive = mbar_wait(empty_bar + 8 * s, (((uint32_t)(kb / TC_STAGES)) & 1u) ^ 1u, abort_flag, status);
            alive = __all_sync(0xffffffffu, alive);
            if (!alive) break;
            tc_fence_after();
            const unsigned char *raw = smem_gen + (size_t)rs * TC_TILE;
            const uint32_t a_col = tmem_a0 + lane_base + (uint32_t)(s * 64);
            uint32_t signs = 0u;
#pragma unroll
            for (int c8 = 0; c8 < 4; ++c8) {                     // 8 contraction indices at a time
                float in[8];
                if (!TRANS) {                                    // chunk c of row r sits at position c ^ (r & 7)
                    const float4 v0 = *reinterpret_cast<const float4 *>(raw + r * 128 + (((2 * c8) ^ (r & 7)) << 4));
                    const float4 v1 = *reinterpret_cast<const float4 *>(raw + r * 128 + (((2 * c8 + 1) ^ (r & 7)) << 4));
                    in[0] = v0.x; in[1] = v0.y; in[2] = v0.z; in[3] = v0.w; in[4] = v1.x; in[5] = v1.y; in[6] = v1.z; in[7] = v1.w;
                } else {                                         // [32 rows of Z][128 columns]
#pragma unroll
                    for (int u = 0; u < 8; ++u) in[u] = reinterpret_cast<const float *>(raw)[(8 * c8 + u) * 128 + r];
                }
                uint32_t h[8], l[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    float e;
                    if (WRITE_MASK) signs |= (in[u] < 0.f ? 1u : 0u) << (8 * c8 + u);
                    if (!MASKED) e = fabsf(in[u]);
                    else if (!TRANS) e = __uint_as_float(__float_as_uint(in[u]) ^ (((word >> (8 * c8 + u)) & 1u) << 31));
                    else e = __uint_as_float(__float_as_uint(in[u]) ^ (((__shfl_sync(0xffffffffu, word, 8 * c8 + u) >> lane) & 1u) << 31));
                    tf32_split(e, h[u], l[u]);
                }
                tmem_st8(a_col + (uint32_t)(8 * c8), h);
                tmem_st8(a_col + (uint32_t)(32 + 8 * c8), l);
            }
            if (WRITE_MASK && row0 + r < p) S_out[(size_t)(row0 + r) * nwords + kb0 + kb] = signs;
            __syncwarp();
            if (lane == 0) mbar_arrive(raw_empty + 8 * rs);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(full_bar + 8 * s);
            word = word_next;
        }
        if (warp < 4) {
            const int grow = row0 + r;
            if (alive) alive = mbar_wait(accum_bar, 0u, abort_flag, status);
            alive = __all_sync(0xffffffffu, alive);
            tc_fence_after();
            float y[LPP];
#pragma unroll
            for (int t = 0; t < LPP; ++t) y[t] = 0.f;
            if (alive && nkb > 0) {
#pragma unroll
                for (int c16 = 0; c16 < (N1 + N2) / 16; ++c16) {
                    uint32_t d[16];
                    tmem_ld16(tmem + lane_base + (uint32_t)(c16 * 16), d);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 16; ++e) y[(c16 * 16 + e) % LPP] += __uint_as_float(d[e]);      // columns t, LPP + t and N1 + t belong to mode t
                }
            }
            if (grow < m_ext) {
                float *out = P + ((size_t)by * m_ext + grow) * LP;
#pragma unroll
                for (int t = 0; t < LP; ++t) out[t] = alive ? y[t] : __int_as_float(0x7fc00000);
            }
        }
    } else if (warp == TC_W_ISSUE || warp == TC_W_ISSUE + 1) {
        // ================================== MMA issuers ===================================
        const bool first = warp == TC_W_ISSUE;                   // first: D1 = E_hi [q_hi | q_lo]; second: D2 = E_lo q_hi
        if (lane == 0) {
            const uint32_t idesc = make_idesc_tf32(first ? N1 : N2);
            const uint32_t d_tmem = tmem + (first ? 0u : (uint32_t)N1);
            bool alive = true;
            for (int kb = 0; kb < nkb && alive; ++kb) {
                const int s = kb % TC_STAGES;
                alive = mbar_wait(full_bar + 8 * s, ((uint32_t)(kb / TC_STAGES)) & 1u, abort_flag, status);
                if (!alive) break;
                tc_fence_after();
                const uint32_t a_t = tmem_a0 + (uint32_t)(s * 64) + (first ? 0u : 32u);
                const uint64_t bdesc = make_smem_desc(img_base + (uint32_t)(s * C::IMG));
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)                   // 8 TF32 per K step: 8 TMEM columns of A, 32 bytes of B
                    umma_ts_tf32(d_tmem, a_t + (uint32_t)(8 * ks), bdesc + (uint64_t)(2 * ks), idesc, (kb > 0 || ks > 0) ? 1u : 0u);
                umma_commit(empty_bar + 8 * s);                  // frees the A stage and the image together
            }
            if (alive && nkb > 0) umma_commit(accum_bar);
            else mbar_arrive(accum_bar);
        }
        __syncwarp();
    } else if (warp == TC_W_RAW) {
        // ================================ raw tile loader ================================
        if (lane == 0) {
            bool alive = true;
            for (int kb = 0; kb < nkb && alive; ++kb) {
                const int rs = kb % TC_RAW;
                alive = mbar_wait(raw_empty + 8 * rs, (((uint32_t)(kb / TC_RAW)) & 1u) ^ 1u, abort_flag, status);
                if (!alive) break;
                mbar_arrive_expect_tx(raw_full + 8 * rs, (uint32_t)TC_TILE);
                if (TRANS) tma_load_2d(smem_base + (uint32_t)(rs * TC_TILE), &tmap_z, row0, (kb0 + kb) * TC_KB, raw_full + 8 * rs);
                else tma_load_2d(smem_base + (uint32_t)(rs * TC_TILE), &tmap_z, (kb0 + kb) * TC_KB, row0, raw_full + 8 * rs);
            }
        }
        __syncwarp();
    } else if (warp == TC_W_IMG) {
        // ================================= image loader ==================================
        if (lane == 0) {
            bool alive = true;
            for (int kb = 0; kb < nkb && alive; ++kb) {
                const int s = kb % TC_STAGES;
                alive = mbar_wait(empty_bar + 8 * s, (((uint32_t)(kb / TC_STAGES)) & 1u) ^ 1u, abort_flag, status);
                if (!alive) break;
                mbar_arrive_expect_tx(full_bar + 8 * s, (uint32_t)C::IMG);
                bulk_load(img_base + (uint32_t)(s * C::IMG), img + (size_t)(kb0 + kb) * (C::IMG / 4), (uint32_t)C::IMG, full_bar + 8 * s);
            }
        }
        __syncwarp();
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) drain_delay();                              // let copies in flight land before the shared memory goes back
    if (warp == TC_W_ISSUE) tmem_dealloc(tmem, (uint32_t)C::TMEM_COLS);
}

// ------------------------------------------------------------------ W = |Z|^T Y
// CTA = 256 columns (thread = column) x a chunk of 256 rows; the chunk's rows of Y sit in shared memory and are read
// by all threads at once (broadcast).  Partial sums per chunk go to P[chunk][column][LP]; a second kernel adds the
// chunks in order (no atomics: the result does not depend on scheduling).
constexpr int ZY_COLS = 256, ZY_ROWS = 256;
template <int LP, bool MASKED>
__global__ void __launch_bounds__(ZY_COLS) abszT_y_kernel(const float *__restrict__ Z, int p, int q, const float *__restrict__ Y,
                                                           float *__restrict__ P, const uint32_t *__restrict__ S, int nwords) {
    __shared__ float Ys[ZY_ROWS][LP];
    const int j = blockIdx.x * ZY_COLS + threadIdx.x;
    const int i0 = blockIdx.y * ZY_ROWS;
    const int nrows = min(ZY_ROWS, p - i0);
    for (int e = threadIdx.x; e < ZY_ROWS * LP; e += ZY_COLS) {
        const int i = e / LP, t = e - i * LP;
        Ys[i][t] = i < nrows ? Y[(size_t)(i0 + i) * LP + t] : 0.f;
    }
    __syncthreads();
    float acc[LP];
#pragma unroll
    for (int t = 0; t < LP; ++t) acc[t] = 0.f;
    if (j < q) {
        const float *zp = Z + (size_t)i0 * q + j;
        const uint32_t *sp = MASKED ? S + (size_t)i0 * nwords + (j >> 5) : nullptr;      // the lanes of a warp share each word
        auto envelope = [&](int i) {
            const float v = zp[(size_t)i * q];
            return MASKED ? __uint_as_float(__float_as_uint(v) ^ (((sp[(size_t)i * nwords] >> (j & 31)) & 1u) << 31)) : fabsf(v);
        };
        int i = 0;
        for (; i + 8 <= nrows; i += 8) {
            float z[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) z[u] = envelope(i + u);
#pragma unroll
            for (int u = 0; u < 8; ++u)
#pragma unroll
                for (int t = 0; t < LP; ++t) acc[t] = fmaf(z[u], Ys[i + u][t], acc[t]);
        }
        for (; i < nrows; ++i) {
            const float z = envelope(i);
#pragma unroll
            for (int t = 0; t < LP; ++t) acc[t] = fmaf(z, Ys[i][t], acc[t]);
        }
        float *out = P + ((size_t)blockIdx.y * q + j) * LP;
#pragma unroll
        for (int t = 0; t < LP; ++t) out[t] = acc[t];
    }
}
__global__ void chunk_sum_kernel(const float *__restrict__ P, int nchunks, size_t n, float *__restrict__ out) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float v = 0.f;
        for (int c = 0; c < nchunks; ++c) v += P[(size_t)c * n + i];
        out[i] = v;
    }
}

// ------------------------------------------------------------------ orth(): Cholesky QR, Gram matrix in fp64
// One warp, lane k = row k of G in registers: G = L L^T (G: the summed Gram matrix, lower triangle), then lane k = column k
// of L^-1 by forward substitution; rows of L travel by shuffles.  M[b][a] = (L^-1)[a][b], so that A M has orthonormal
// columns.  A zero (or numerically vanished) pivot - a padding column, or a block wider than the rank of the matrix -
// leaves its column as it is instead of dividing by zero.
template <int LP>
__device__ __forceinline__ void chol_warp(const double (*Gm)[LP + 1], float *__restrict__ M) {
    const int k = threadIdx.x & 31;
    double g[LP], invd[LP];
    double scale = 0.0;
#pragma unroll
    for (int j = 0; j < LP; ++j) {
        g[j] = (k < LP && j <= k) ? Gm[k < LP ? k : 0][j] : 0.0;
        scale = fmax(scale, Gm[j][j]);
    }
#pragma unroll
    for (int c = 0; c < LP; ++c) {
        const double dcc = __shfl_sync(0xffffffffu, g[c], c);
        const double inv = (dcc > 1e-24 * scale && dcc > 0.0) ? rsqrt(dcc) : 0.0;
        invd[c] = inv;                                           // 1 / L[c][c], the same in every lane
        g[c] = k == c ? dcc * inv : g[c] * inv;                  // column c of L (zero above the diagonal)
#pragma unroll
        for (int jj = c + 1; jj < LP; ++jj) {
            const double ljc = __shfl_sync(0xffffffffu, g[c], jj);
            if (k >= jj) g[jj] -= g[c] * ljc;
        }
    }
    double x[LP];
#pragma unroll
    for (int i = 0; i < LP; ++i) {
        double sum = i == k ? 1.0 : 0.0;
#pragma unroll
        for (int m = 0; m < i; ++m) {
            const double lim = __shfl_sync(0xffffffffu, g[m], i);     // L[i][m]
            if (m >= k) sum -= lim * x[m];
        }
        x[i] = i >= k ? (invd[i] > 0.0 ? sum * invd[i] : (i == k ? 1.0 : 0.0)) : 0.0;
    }
    if (k < LP) {
#pragma unroll
        for (int a = 0; a < LP; ++a) M[k * LP + a] = (float)x[a];
    }
}
// Gram matrix of a tall matrix A (n x LP) in fp64 and what follows it, in one launch.  The CTAs stride over chunks of
// GR_ROWS rows: where `parts` > 0 a chunk's rows are first formed as the sum of their partial sums P[c] (c < parts, in
// order) and written to A; every CTA keeps one partial Gram matrix (lower triangle) over its chunks.  The CTA that
// finishes last adds the CTAs' matrices up in a fixed order and either factors the sum (CHOL: M for right_mul_kernel)
// or leaves it in Gs for the eigensolver.
constexpr int GR_ROWS = 128, GR_MAX_CTAS = 128;
template <int LP, bool CHOL>
__global__ void __launch_bounds__(256) gram_finish_kernel(float *__restrict__ A, int n, const float *__restrict__ P, int parts,
                                                          double *__restrict__ Gp, unsigned int *__restrict__ counter,
                                                          double *__restrict__ Gs, float *__restrict__ M) {
    constexpr int PER = GR_ROWS * LP / 256 > 0 ? GR_ROWS * LP / 256 : 1;     // elements of a chunk per thread
    constexpr int ENT = (LP * LP + 255) / 256;                                // Gram entries per thread
    __shared__ double As[GR_ROWS][LP + 1];                       // converted once on the way in, not once per product
    __shared__ double Gm[LP][LP + 1];
    __shared__ bool is_last;
    double acc[ENT];
#pragma unroll
    for (int u = 0; u < ENT; ++u) acc[u] = 0.0;
    const int nchunks = (n + GR_ROWS - 1) / GR_ROWS;
    for (int chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
        const int i0 = chunk * GR_ROWS;
        const size_t base = (size_t)i0 * LP, limit = (size_t)n * LP;
        float v[PER];
#pragma unroll
        for (int u = 0; u < PER; ++u) v[u] = 0.f;
        if (parts > 0) {
#pragma unroll 4
            for (int c = 0; c < parts; ++c)                       // independent loads, additions in the order of c
#pragma unroll
                for (int u = 0; u < PER; ++u) {
                    const size_t at = base + threadIdx.x + 256 * u;
                    if (threadIdx.x + 256 * u < GR_ROWS * LP && at < limit) v[u] += __ldcs(P + (size_t)c * limit + at);
                }
        } else {
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                const size_t at = base + threadIdx.x + 256 * u;
                if (threadIdx.x + 256 * u < GR_ROWS * LP && at < limit) v[u] = A[at];
            }
        }
        __syncthreads();                                         // the previous chunk's Gram pass has read As
#pragma unroll
        for (int u = 0; u < PER; ++u) {
            const int e = threadIdx.x + 256 * u;
            if (e < GR_ROWS * LP) {
                const size_t at = base + e;
                if (parts > 0 && at < limit) A[at] = v[u];
                As[e / LP][e % LP] = (double)v[u];               // rows past the end are zero
            }
        }
        __syncthreads();
#pragma unroll
        for (int u = 0; u < ENT; ++u) {
            const int pr = threadIdx.x + 256 * u;
            const int a = pr / LP, b = pr - a * LP;
            if (pr < LP * LP && b <= a) {
                double s0 = 0.0, s1 = 0.0;
                for (int i = 0; i < GR_ROWS; i += 2) {
                    s0 += As[i][a] * As[i][b];
                    s1 += As[i + 1][a] * As[i + 1][b];
                }
                acc[u] += s0 + s1;
            }
        }
    }
#pragma unroll
    for (int u = 0; u < ENT; ++u)
        if (threadIdx.x + 256 * u < LP * LP) Gp[(size_t)blockIdx.x * LP * LP + threadIdx.x + 256 * u] = acc[u];
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = atomicAdd(counter, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int pr = threadIdx.x; pr < LP * LP; pr += 256) {
        double s[4] = {0.0, 0.0, 0.0, 0.0};
        for (int c = 0; c < (int)gridDim.x; c += 16) {           // sixteen loads in flight, added in the order of c
            double v[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) v[u] = c + u < (int)gridDim.x ? __ldcg(Gp + (size_t)(c + u) * LP * LP + pr) : 0.0;
#pragma unroll
            for (int u = 0; u < 16; ++u) s[u & 3] += v[u];
        }
        const double total = (s[0] + s[1]) + (s[2] + s[3]);
        if (CHOL) Gm[pr / LP][pr % LP] = total;
        else Gs[pr] = total;
    }
    if (threadIdx.x == 0) *counter = 0u;                         // ready for the next launch on the stream
    if (!CHOL) return;
    __syncthreads();
    if (threadIdx.x < 32) chol_warp<LP>(Gm, M);
}
// A <- A M, row by row (M is LP x LP, row-major).  With `img`, the rows' operand images for the tensor-core product that
// reads A next are written on the way out: per block of 32 rows (= 32 contraction indices kappa) a tile of 2 LPP rows of
// 32 TF32 values, 128 bytes each, 16-byte chunk c of row r at position c ^ (r & 7) (the 128B swizzle of a K-major
// operand); row t < LPP holds the TF32 rounding of column t, row LPP + t the rounded residual; rows past the end are zero.
template <int LP>
__global__ void __launch_bounds__(256) right_mul_kernel(float *__restrict__ A, int n, const float *__restrict__ M, float *__restrict__ out,
                                                        int out_cols, uint32_t *__restrict__ img) {
    __shared__ float Ms[LP][LP];
    for (int e = threadIdx.x; e < LP * LP; e += 256) Ms[e / LP][e % LP] = M[e];
    __syncthreads();
    const int i = blockIdx.x * 256 + threadIdx.x;
    float a[LP], o[LP];
#pragma unroll
    for (int t = 0; t < LP; ++t) { a[t] = i < n ? A[(size_t)i * LP + t] : 0.f; o[t] = 0.f; }
#pragma unroll
    for (int b = 0; b < LP; ++b)
#pragma unroll
        for (int t = 0; t < LP; ++t) o[t] = fmaf(a[b], Ms[b][t], o[t]);
    if (img && i < ((n + TC_KB - 1) / TC_KB) * TC_KB) {
        constexpr int LPP = TcCfg<LP>::LPP, N1 = TcCfg<LP>::N1;
        const int kappa = i & 31;
        uint32_t *dst = img + (size_t)(i >> 5) * (N1 * 32);
#pragma unroll
        for (int t = 0; t < LPP; ++t) {
            const float v = t < LP ? o[t < LP ? t : 0] : 0.f;
            const uint32_t hi = tf32_round(v);
            dst[t * 32 + ((((kappa >> 2) ^ (t & 7)) << 2) | (kappa & 3))] = hi;
            dst[(LPP + t) * 32 + ((((kappa >> 2) ^ ((LPP + t) & 7)) << 2) | (kappa & 3))] = tf32_round(v - __uint_as_float(hi));
        }
    }
    if (i >= n) return;
    if (out) {
        for (int t = 0; t < out_cols; ++t) out[(size_t)i * out_cols + t] = o[t];     // compact result (the first out_cols columns)
    } else {
#pragma unroll
        for (int t = 0; t < LP; ++t) A[(size_t)i * LP + t] = o[t];
    }
}

// ------------------------------------------------------------------ the small eigenproblem
// One CTA: Jacobi on G = Y^T Y (l x l, fp64, given as its lower triangle), eigenvalues sorted in descending order;
// writes the singular values s_t = sqrt(lambda_t) and the two LP x LP matrices that turn (Y, Q) into the balanced
// factors: MU[b][t] = W[b][t] s_t^-1/2, MV[b][t] = W[b][t] s_t^1/2 (zero columns beyond l and for vanished values).
// Round-robin ordering: n - 1 rounds of n / 2 rotations on disjoint index pairs (n = l rounded up to even; a pair with
// the dummy index is skipped).  Thread i < n / 2 works out the rotation of pair i; then thread (k, i) applies rotation
// i to row k (columns p, q of G and of W), and after a barrier to column k (rows p, q of G).  The tangent is taken in
// fp32 (any angle near the optimal one converges; fp64 division and square roots were most of a round), the cosine
// and sine from it in fp64, so that every rotation is orthogonal to fp64 rounding.
constexpr int JAC_THREADS = 256;
template <int LP>
__global__ void __launch_bounds__(JAC_THREADS) jacobi_kernel(const double *__restrict__ Gs, int l, float *__restrict__ sigma,
                                                             float *__restrict__ MU, float *__restrict__ MV) {
    __shared__ double G[LP][LP + 1], W[LP][LP + 1], rc[LP], rs[LP];
    __shared__ int order[LP], rp[LP], rq[LP];
    __shared__ int done;
    const int tid = threadIdx.x;
    for (int e = tid; e < LP * LP; e += JAC_THREADS) {
        const int a = e / LP, b = e - a * LP;
        G[a][b] = Gs[b <= a ? a * LP + b : b * LP + a];
        W[a][b] = a == b ? 1.0 : 0.0;
    }
    const int n = (l + 1) & ~1, half = n / 2;
    for (int sweep = 0; sweep < 30 && n >= 2; ++sweep) {
        __syncthreads();
        if (tid < 32) {
            double off = 0.0, diag = 0.0;
            for (int k = tid; k < l; k += 32) {
                diag += G[k][k] * G[k][k];
                for (int b = 0; b < k; ++b) off += G[k][b] * G[k][b];
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                off += __shfl_xor_sync(0xffffffffu, off, o);
                diag += __shfl_xor_sync(0xffffffffu, diag, o);
            }
            if (tid == 0) done = off <= 1e-20 * diag;            // off-diagonal mass below 1e-10 of the diagonal's: the eigenvalues are
                                                                 // then accurate to the square of that
        }
        __syncthreads();
        if (done) break;
        for (int r = 0; r < n - 1; ++r) {
            if (tid < half) {
                const int a = tid == 0 ? n - 1 : (r + tid) % (n - 1), b = tid == 0 ? r : (r - tid + (n - 1)) % (n - 1);
                const int pi = min(a, b), qi = max(a, b);
                double c = 1.0, sn = 0.0;
                if (qi < l) {
                    const double apq = G[pi][qi];
                    if (apq != 0.0) {
                        const float theta = (float)(G[qi][qi] - G[pi][pi]) / (2.f * (float)apq);
                        const double t = (double)((theta >= 0.f ? 1.f : -1.f) / (fabsf(theta) + sqrtf(theta * theta + 1.f)));
                        c = rsqrt(t * t + 1.0);
                        sn = t * c;
                    }
                }
                rp[tid] = pi; rq[tid] = qi; rc[tid] = c; rs[tid] = sn;
            }
            __syncthreads();
            for (int idx = tid; idx < l * half; idx += JAC_THREADS) {
                const int k = idx / half, i = idx - k * half;
                const double c = rc[i], sn = rs[i];
                if (sn == 0.0) continue;
                const int pi = rp[i], qi = rq[i];
                const double gkp = G[k][pi], gkq = G[k][qi];
                G[k][pi] = c * gkp - sn * gkq;
                G[k][qi] = sn * gkp + c * gkq;
                const double wkp = W[k][pi], wkq = W[k][qi];
                W[k][pi] = c * wkp - sn * wkq;
                W[k][qi] = sn * wkp + c * wkq;
            }
            __syncthreads();
            for (int idx = tid; idx < l * half; idx += JAC_THREADS) {
                const int k = idx / half, i = idx - k * half;
                const double c = rc[i], sn = rs[i];
                if (sn == 0.0) continue;
                const int pi = rp[i], qi = rq[i];
                const double gpk = G[pi][k], gqk = G[qi][k];
                G[pi][k] = c * gpk - sn * gqk;
                G[qi][k] = sn * gpk + c * gqk;
            }
            __syncthreads();
        }
    }
    __syncthreads();
    if (tid == 0) {
        for (int t = 0; t < l; ++t) order[t] = t;
        for (int t = 0; t < l; ++t)                    // selection sort, descending eigenvalues
            for (int u = t + 1; u < l; ++u)
                if (G[order[u]][order[u]] > G[order[t]][order[t]]) { const int x = order[t]; order[t] = order[u]; order[u] = x; }
    }
    __syncthreads();
    const double top = l > 0 ? fmax(G[order[0]][order[0]], 0.0) : 0.0;
    for (int e = tid; e < LP * LP; e += JAC_THREADS) {
        const int k = e / LP, t = e - k * LP;
        double lam = t < l ? G[order[t]][order[t]] : 0.0;
        if (!(lam > 1e-24 * top)) lam = 0.0;
        const double sv = sqrt(lam), rsv = sqrt(sv);
        if (k == 0 && t < l) sigma[t] = (float)sv;
        const double w = (t < l && k < l) ? W[k][order[t]] : 0.0;
        MU[k * LP + t] = (float)(rsv > 0.0 ? w / rsv : 0.0);
        MV[k * LP + t] = (float)(w * rsv);
    }
}

// start block: Q0 (M x l, compact) -> Q (M x LP, zero padding)
__global__ void pad_kernel(const float *__restrict__ src, size_t n, int l, int LP, float *__restrict__ dst) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n * LP; e += (size_t)gridDim.x * blockDim.x) {
        const size_t i = e / LP;
        const int t = (int)(e - i * LP);
        dst[e] = t < l ? src[i * l + t] : 0.f;
    }
}

// The scratch of one call, carved out of the caller's workspace (256-byte aligned pieces).
struct Scratch {
    float *Q, *Y, *P, *M, *MU, *MV;
    double *Gp, *Gs;
    uint32_t *img;          // operand images of Q for the tensor-core product
    int32_t *status;        // set by a wait that ran out
    unsigned int *counter;  // CTAs of the Gram kernel that have finished (the word after the status word)
};
// how the K blocks of the tensor-core product are split over blockIdx.y: the split that fills whole waves of resident CTAs best,
// each CTA keeping at least 8 K blocks
static int tc_split(int p, int q, int LP, int *kb_per_cta) {
    const int slots = 148 * 2;                                   // two CTAs per SM
    (void)LP;
    const int rb = ceil_div(p, 128), nkb = ceil_div(q, TC_KB);
    int best = 1;
    double best_eff = -1.0;
    for (int ns = 1; ns <= 16 && nkb / ns >= 8; ++ns) {
        const int per = ceil_div(nkb, ns), parts = ceil_div(nkb, per);
        const int ctas = rb * parts, waves = ceil_div(ctas, slots);
        const double eff = (double)rb * nkb / ((double)waves * slots * per);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = ns; }
    }
    *kb_per_cta = ceil_div(nkb, best);
    return ceil_div(nkb, *kb_per_cta);
}
static size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }
static size_t carve(Scratch *w, char *base, int p, int q, int LP) {
    const size_t zy_chunks = ceil_div(p, ZY_ROWS), gchunks = GR_MAX_CTAS;
    size_t off = 0;
    auto take = [&](size_t bytes) { char *ptr = base ? base + off : nullptr; off += align256(bytes); return ptr; };
    float *Q = (float *)take((size_t)q * LP * sizeof(float));
    float *Y = (float *)take((size_t)p * LP * sizeof(float));
    int kb_per_cta = 0;
    const size_t tc_parts = (size_t)tc_split(p, q, LP, &kb_per_cta), tc_parts_t = (size_t)tc_split(q, p, LP, &kb_per_cta);
    float *P = (float *)take(std::max(std::max(zy_chunks, tc_parts_t) * q, tc_parts * p) * LP * sizeof(float));
    uint32_t *img = (uint32_t *)take((size_t)ceil_div(std::max(p, q), TC_KB) * 2 * (LP < 16 ? 16 : LP) * 128);
    int32_t *status = (int32_t *)take(2 * sizeof(int32_t));
    double *Gp = (double *)take(gchunks * LP * LP * sizeof(double));
    double *Gs = (double *)take((size_t)LP * LP * sizeof(double));
    float *M = (float *)take((size_t)LP * LP * sizeof(float));
    float *MU = (float *)take((size_t)LP * LP * sizeof(float));
    float *MV = (float *)take((size_t)LP * LP * sizeof(float));
    if (w) { w->Q = Q; w->Y = Y; w->P = P; w->Gp = Gp; w->Gs = Gs; w->M = M; w->MU = MU; w->MV = MV; w->img = img; w->status = status; w->counter = (unsigned int *)status + 1; }
    return off;
}
static int padded_rank(int l) {
    int LP = 1;
    while (LP < l) LP *= 2;
    return LP;
}

// A <- an orthonormal basis of its columns (Cholesky QR); with `parts` > 0, A is first formed as the sum of the partial sums
// in w.P; with `img`, the operand images of the result are written for the tensor-core product that reads it next
template <int LP>
static mdbf_status_t orth(float *A, int n, Scratch &w, cudaStream_t st, int parts = 0, uint32_t *img = nullptr) {
    gram_finish_kernel<LP, true><<<std::min(ceil_div(n, GR_ROWS), GR_MAX_CTAS), 256, 0, st>>>(A, n, w.P, parts, w.Gp, w.counter, w.Gs, w.M);
    right_mul_kernel<LP><<<ceil_div(n, 256), 256, 0, st>>>(A, n, w.M, nullptr, 0, img);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

// Tensor map of the fp32 matrix Z [p][q]: box of box_cols columns x box_rows rows, zero fill outside the matrix.
static mdbf_status_t make_z_tensor_map(CUtensorMap *out, const float *Z, int p, int q, int box_cols, int box_rows, bool swizzle128) {
    typedef CUresult (*encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static encode_fn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult res;
        MDBF_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &res));
        if (!ptr || res != cudaDriverEntryPointSuccess) {
            set_error("cuTensorMapEncodeTiled is not available from the driver");
            return MDBF_ERR_CUDA;
        }
        fn = reinterpret_cast<encode_fn>(ptr);
    }
    const cuuint64_t gdim[2] = {(cuuint64_t)q, (cuuint64_t)p};
    const cuuint64_t gstride[1] = {(cuuint64_t)q * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(Z), gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled (Z) failed with CUresult %d", (int)r);
        return MDBF_ERR_CUDA;
    }
    return MDBF_OK;
}
static bool tc_eligible(const float *Z, int q) { return (q & 3) == 0 && (reinterpret_cast<uintptr_t>(Z) & 15u) == 0; }

struct ZMaps {
    bool use;               // the tensor-core kernels run (else the scalar ones)
    CUtensorMap rows;       // box of 32 columns x 128 rows, 128B swizzle, for Y = E Q
    CUtensorMap cols;       // box of 128 columns x 32 rows, for W = E^T Y
};
// E F (TRANS = false: p output rows, F has q) or E^T F (TRANS = true: q output rows, F has p) on the tensor cores, E the
// envelope of Z (|Z|, or Z with the given mask's signs taken off) and F the factor whose operand images the preceding
// right_mul_kernel left in w.img; the result is left as *parts_out partial sums in w.P
template <int LP, bool MASKED, bool TRANS, bool WRITE_MASK = false>
static mdbf_status_t tc_product(const ZMaps &zm, int p, int q, const uint32_t *S, int nwords, Scratch &w,
                                cudaStream_t st, int *parts_out, uint32_t *S_out = nullptr) {
    using C = TcCfg<LP>;
    static PerDeviceOnce once;
    if (once.first())
        MDBF_CUDA(cudaFuncSetAttribute(envelope_product_tc_kernel<LP, MASKED, TRANS, WRITE_MASK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)C::SMEM));
    const int m_ext = TRANS ? q : p, k_ext = TRANS ? p : q;
    int kb_per_cta = 0;
    const int parts = tc_split(m_ext, k_ext, LP, &kb_per_cta);
    envelope_product_tc_kernel<LP, MASKED, TRANS, WRITE_MASK><<<dim3(ceil_div(m_ext, 128), parts), TC_THREADS, C::SMEM, st>>>(
        TRANS ? zm.cols : zm.rows, p, q, w.img, kb_per_cta, w.P, S, S_out, nwords, w.status);
    *parts_out = parts;                                          // the Gram kernel that follows adds the partial sums up
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}
// Y = E Q
template <int LP, bool MASKED>
static mdbf_status_t product(const float *Z, int p, int q, const uint32_t *S, int nwords, const ZMaps &zm, Scratch &w, cudaStream_t st,
                             int *parts, uint32_t *S_out = nullptr) {
    if (zm.use) {
        if constexpr (!MASKED)
            if (S_out) return tc_product<LP, false, false, true>(zm, p, q, S, nwords, w, st, parts, S_out);
        return tc_product<LP, MASKED, false>(zm, p, q, S, nwords, w, st, parts);
    }
    *parts = 0;                                                  // the scalar kernels write the whole result
    absz_q_kernel<LP, MASKED><<<ceil_div(p, AQ_WARPS * AQ_ROWS), AQ_WARPS * 32, 0, st>>>(Z, p, q, w.Q, w.Y, S, nwords);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}
// Q = E^T Y
template <int LP, bool MASKED>
static mdbf_status_t product_t(const float *Z, int p, int q, const uint32_t *S, int nwords, const ZMaps &zm, Scratch &w, cudaStream_t st,
                               int *parts) {
    if (zm.use && LP >= 8) return tc_product<LP, MASKED, true>(zm, p, q, S, nwords, w, st, parts);
    *parts = 0;   // narrower blocks: the scalar kernel runs at the memory rate already
    const int zy_chunks = ceil_div(p, ZY_ROWS);
    abszT_y_kernel<LP, MASKED><<<dim3(ceil_div(q, ZY_COLS), zy_chunks), ZY_COLS, 0, st>>>(Z, p, q, w.Y, w.P, S, nwords);
    chunk_sum_kernel<<<(int)std::min<size_t>(((size_t)q * LP + 255) / 256, 148u * 8), 256, 0, st>>>(w.P, zy_chunks, (size_t)q * LP, w.Q);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

// MASKED = false: S is written (the mask of Z itself, Eq. msvid-def); MASKED = true: S is given (Eq. Ustar)
template <int LP, bool MASKED>
static mdbf_status_t run(const float *Z, int p, int q, int l, int n_iter, const float *Q0, uint32_t *S, float *U, float *V, float *sigma,
                         Scratch &w, cudaStream_t st) {
    const int nwords = ceil_div(q, 32);
    MDBF_CUDA(cudaMemsetAsync(w.status, 0, 2 * sizeof(int32_t), st));           // status word and the Gram kernel's counter
    ZMaps zm;
    zm.use = tc_eligible(Z, q);
    if (zm.use) {
        mdbf_status_t rcm = make_z_tensor_map(&zm.rows, Z, p, q, TC_KB, 128, true);
        if (rcm == MDBF_OK) rcm = make_z_tensor_map(&zm.cols, Z, p, q, 128, TC_KB, false);
        if (rcm) return rcm;
    }
    // the mask of Z itself: packed by the first tensor-core pass over Z, else by a pass of its own
    if (!MASKED && !zm.use) sign_pack_kernel<<<dim3(p, ceil_div(nwords, 8 * SP_WORDS)), 256, 0, st>>>(Z, q, nwords, S);
    pad_kernel<<<(int)std::min<size_t>(((size_t)q * LP + 255) / 256, 148u * 8), 256, 0, st>>>(Q0, (size_t)q, l, LP, w.Q);
    MDBF_CUDA(cudaGetLastError());
    mdbf_status_t rc = orth<LP>(w.Q, q, w, st);                        // twice: the start block may be badly conditioned
    uint32_t *img_q = zm.use ? w.img : nullptr, *img_y = (zm.use && LP >= 8) ? w.img : nullptr;   // which products run on the tensor cores
    if (rc == MDBF_OK) rc = orth<LP>(w.Q, q, w, st, 0, img_q);
    if (rc) return rc;
    int parts = 0;
    for (int it = 0; it < n_iter; ++it) {
        rc = product<LP, MASKED>(Z, p, q, S, nwords, zm, w, st, &parts, (!MASKED && it == 0) ? S : nullptr);
        if (rc == MDBF_OK) rc = orth<LP>(w.Y, p, w, st, parts, img_y);
        if (rc == MDBF_OK) rc = product_t<LP, MASKED>(Z, p, q, S, nwords, zm, w, st, &parts);
        if (rc == MDBF_OK) rc = orth<LP>(w.Q, q, w, st, parts, it == n_iter - 1 ? nullptr : img_q);
        if (rc == MDBF_OK && it == n_iter - 1) rc = orth<LP>(w.Q, q, w, st, 0, img_q);   // the last block carries the result: orthonormal to fp32
        if (rc) return rc;
    }
    rc = product<LP, MASKED>(Z, p, q, S, nwords, zm, w, st, &parts);
    if (rc) return rc;
    gram_finish_kernel<LP, false><<<std::min(ceil_div(p, GR_ROWS), GR_MAX_CTAS), 256, 0, st>>>(w.Y, p, w.P, parts, w.Gp, w.counter, w.Gs, w.M);
    jacobi_kernel<LP><<<1, JAC_THREADS, 0, st>>>(w.Gs, l, sigma, w.MU, w.MV);
    right_mul_kernel<LP><<<ceil_div(p, 256), 256, 0, st>>>(w.Y, p, w.MU, U, l, nullptr);
    right_mul_kernel<LP><<<ceil_div(q, 256), 256, 0, st>>>(w.Q, q, w.MV, V, l, nullptr);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

static mdbf_status_t check_shape(const char *who, int64_t rows, int64_t cols, int32_t l) {
    if (rows < 1 || cols < 1 || rows > (1 << 24) || cols > (1 << 24) || rows * cols > (1LL << 40)) {
        set_error("%s: size %lld x %lld outside the supported range", who, (long long)rows, (long long)cols);
        return MDBF_ERR_SHAPE;
    }
    if (l < 1 || l > kMaxL || l > rows || l > cols) {
        set_error("%s: l=%d outside [1, min(%d, rows, cols)]", who, l, kMaxL);
        return MDBF_ERR_SHAPE;
    }
    return MDBF_OK;
}

}  // namespace msv
}  // namespace mdbf

using namespace mdbf;

extern "C" mdbf_status_t mdbf_msvid_workspace_bytes(int64_t rows, int64_t cols, int32_t l, size_t *bytes) {
    if (!bytes) { set_error("mdbf_msvid_workspace_bytes: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    mdbf_status_t rc = msv::check_shape("mdbf_msvid_workspace_bytes", rows, cols, l);
    if (rc) return rc;
    *bytes = msv::carve(nullptr, nullptr, (int)rows, (int)cols, msv::padded_rank(l));
    return MDBF_OK;
}

static mdbf_status_t msvid_entry(const char *who, bool masked, const float *Z, int64_t rows, int64_t cols, int32_t l, int32_t n_iter,
                                 const float *Q0, uint32_t *S_packed, float *U, float *V, float *sigma, void *workspace,
                                 size_t workspace_bytes, void *stream) {
    if (!Z || !Q0 || !S_packed || !U || !V || !sigma || !workspace) { set_error("%s: NULL pointer", who); return MDBF_ERR_INVALID_ARG; }
    mdbf_status_t rc = msv::check_shape(who, rows, cols, l);
    if (rc) return rc;
    if (n_iter < 1 || n_iter > 1000) { set_error("%s: n_iter=%d outside [1, 1000]", who, n_iter); return MDBF_ERR_SHAPE; }
    const int p = (int)rows, q = (int)cols, LP = msv::padded_rank(l);
    msv::Scratch w;
    const size_t need = msv::carve(&w, (char *)workspace, p, q, LP);
    if (workspace_bytes < need || ((uintptr_t)workspace & 255u) != 0) {
        set_error("%s: the workspace must hold %zu bytes (mdbf_msvid_workspace_bytes) on a 256-byte boundary; got %zu at %p", who,
                  need, workspace_bytes, workspace);
        return MDBF_ERR_INVALID_ARG;
    }
    rc = require_device(nullptr);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
#define MSV_RUN(LPV)                                                                                              \
    return masked ? msv::run<LPV, true>(Z, p, q, l, n_iter, Q0, S_packed, U, V, sigma, w, st)                    \
                  : msv::run<LPV, false>(Z, p, q, l, n_iter, Q0, S_packed, U, V, sigma, w, st)
    switch (LP) {
        case 1: MSV_RUN(1);
        case 2: MSV_RUN(2);
        case 4: MSV_RUN(4);
        case 8: MSV_RUN(8);
        case 16: MSV_RUN(16);
        default: MSV_RUN(32);
    }
#undef MSV_RUN
}

extern "C" mdbf_status_t mdbf_msvid(const float *Z, int64_t rows, int64_t cols, int32_t l, int32_t n_iter, const float *Q0,
                                    uint32_t *S_packed, float *U, float *V, float *sigma, void *workspace, size_t workspace_bytes,
                                    void *stream) {
    return msvid_entry("mdbf_msvid", false, Z, rows, cols, l, n_iter, Q0, S_packed, U, V, sigma, workspace, workspace_bytes, stream);
}

extern "C" mdbf_status_t mdbf_project_fixed_mask(const float *Z, const uint32_t *S_packed, int64_t rows, int64_t cols, int32_t l,
                                                 int32_t n_iter, const float *Q0, float *U, float *V, float *sigma, void *workspace,
                                                 size_t workspace_bytes, void *stream) {
    return msvid_entry("mdbf_project_fixed_mask", true, Z, rows, cols, l, n_iter, Q0, const_cast<uint32_t *>(S_packed), U, V, sigma,
                       workspace, workspace_bytes, stream);
}
