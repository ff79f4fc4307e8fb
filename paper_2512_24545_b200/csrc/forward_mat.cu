// Materialised-envelope evaluation order of the MDBF forward for T >= 2 tokens.
//
// A stage applies  W_hat = S (.) (U V^T)  (Eq. me-dbf-basis: one sign matrix under a rank-l real
// envelope).  Instead of expanding it into l sign GEMMs (Eq. me-dbf-expand, width l*T), this
// kernel rebuilds W_hat tile by tile on the fly and runs ONE GEMM of width T:
//
//     E[r][c]      = sum_t U[r][t] V[c][t]                 rank-l mini-MMA on the tensor core, fp32 in TMEM
//     W_hat[r][c]  = bf16(E[r][c]) with the sign bit flipped where S[r][c] = -1      (CUDA cores)
//     out[tau][r]  = sum_c W_hat[r][c] in[tau][c]          tcgen05.mma, fp32 accumulator in TMEM
//
// Per weight bit it executes 2T + 2*max(l,16) tensor FLOP instead of 2*l*T, needs no pre-scaled
// copies of the activations (the TMA reads x, and the bf16 intermediate z, as they are) and
// two launches per forward.  The result differs from the expanded order only in rounding:
// W_hat is rounded to bf16 once per entry, the activations are not rounded at all.
//
// CTA = 128 rows of W_hat x up to 256 tokens, 12 warps:
//   warps 0-7  two groups of four on alternate K blocks (64 columns).  Per block a thread (= row =
//              TMEM lane) reads its 64 fp32 envelope values with tcgen05.ld, packs pairs to bf16,
//              XORs the sign bits of its 64 packed bits in, and writes the 128B-swizzled A tile.
//              Afterwards both groups run the epilogue on alternate 32-token chunks.
//   warp 8     one lane issues the TMA load of the activation tile [tokens x 64]
//   warp 9     one lane issues the 4 main MMAs of a K block and commits the stage
//   warp 10    one lane bulk-copies the envelope images (U once, V per K block, ring of 6 or 8)
//   warp 11    one lane issues the mini-MMAs (U image x V image, no swizzle) into a ring of four
//              64-column TMEM buffers, as far ahead of the main MMAs as the ring allows.  A warp of
//              its own: one thread's chain of barrier tests, MMAs and commits would otherwise cap
//              the rate of the main MMAs.
// Ring: stages of (A 16 KB + activation tile), 4 deep at 256 tokens per tile and up to 10 deep with
// narrower tiles.  TMEM: 256 accumulator + 4 x 64 envelope columns.
//
// Every mbarrier wait is bounded; when one expires the kernel records MDBF_ERR_TIMEOUT in the
// layer's status word, all roles fall through to the common exit, TMEM is released and the kernel
// returns.  No TMA multicast is used.
#include "tmem_ptx.cuh"

namespace mdbf {

constexpr int MT_BM = 128;
constexpr int MT_BN = 256;
constexpr int MT_BK = 64;
constexpr int MT_STAGES = 4;
constexpr int MT_GROUPS = 2;
constexpr int MT_W_TMA = MT_GROUPS * 4;
constexpr int MT_W_MMA = MT_W_TMA + 1;
constexpr int MT_W_ENV = MT_W_TMA + 2;
constexpr int MT_W_MINI = MT_W_TMA + 3;
constexpr int MT_THREADS = (MT_W_MINI + 1) * 32;
constexpr int MT_A_BYTES = MT_BM * MT_BK * 2;
constexpr int MT_B_BYTES = MT_BN * MT_BK * 2;
constexpr int MT_MAX_NS = 10;            // ring depth: 4 stages at 256 tokens per tile, more with narrower tiles
constexpr int MT_RING_BYTES = MT_STAGES * (MT_A_BYTES + MT_B_BYTES);
constexpr int MT_NE = 4;                 // envelope buffers in TMEM
constexpr int MT_MAX_NV = 8;             // V-image ring depth (8 with l <= 16, 6 with l <= 32)
constexpr int MT_TMEM_COLS = 512;

struct MatArgs {
    const uint2 *wk;         // K-blocked sign words [kblocks][rows_pad], 64 bits per row and block
    int rows_pad;
    int rows, cols;
    const uint16_t *uimg;    // [row block][KC][16][8][8] 16-bit envelope values (see uimg_kernel)
    const uint16_t *vimg;    // [K block][KC][8][8][8]
    int kc;                  // 16-byte chunks of the mode axis: 2 (l <= 16) or 4 (l <= 32)
    uint32_t env_fmt;        // 0: f16 envelopes, 1: bf16
    int nv;                  // V-image ring depth
    int T;
    int bn;                  // tokens per CTA tile = MMA N = rows of the TMA box (multiple of 16, <= 256)
    int ns;                  // ring depth (stages of A tile + activation tile)
    __nv_bfloat16 *zb;       // stage B: bf16 intermediate [T][zstride]
    int zstride;
    __nv_bfloat16 *y;        // stage A: [T][rows]
    float *y32;              // stage A, fp32 output modes (y_mode 1: store, 2: add)
    int y_mode;
    int32_t *status;
};

// --------------------------------------------------------- pack-time envelope images
// U of one row block as the A operand of the mini-MMA (K-major, no swizzle): the 16-bit value of
// row 128*rb + 8*g + i, mode 8*c + e sits at element ((c*16 + g)*8 + i)*8 + e of the block's image.
__global__ void uimg_kernel(const void *__restrict__ U, int rows, int l, int env_dtype, uint16_t *__restrict__ out,
                            int rblocks, int kc) {
    const size_t per = (size_t)kc * 16 * 64;
    const size_t total = (size_t)rblocks * per;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int rb = (int)(idx / per);
        const int rem = (int)(idx % per);
        const int e = rem & 7, i = (rem >> 3) & 7, g = (rem >> 6) & 15, c = rem >> 10;
        const int row = rb * 128 + g * 8 + i, t = c * 8 + e;
        uint16_t v = 0;
        if (row < rows && t < l) v = reinterpret_cast<const uint16_t *>(U)[(size_t)row * l + t];
        out[idx] = v;
    }
}
// V of one K block as the B operand: column 64*kb + 8*g + i, mode 8*c + e at ((c*8 + g)*8 + i)*8 + e.
__global__ void vimg_kernel(const void *__restrict__ V, int cols, int l, int env_dtype, uint16_t *__restrict__ out,
                            int kblocks, int kc) {
    const size_t per = (size_t)kc * 8 * 64;
    const size_t total = (size_t)kblocks * per;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int kb = (int)(idx / per);
        const int rem = (int)(idx % per);
        const int e = rem & 7, i = (rem >> 3) & 7, g = (rem >> 6) & 7, c = rem >> 9;
        const int col = kb * 64 + g * 8 + i, t = c * 8 + e;
        uint16_t v = 0;
        if (col < cols && t < l) v = reinterpret_cast<const uint16_t *>(V)[(size_t)col * l + t];
        out[idx] = v;
    }
}

static int mt_grid(size_t items) {
    size_t g = (items + 255) / 256;
    if (g < 1) g = 1;
    if (g > 148 * 32) g = 148 * 32;
    return (int)g;
}
mdbf_status_t launch_uimg(const void *U, int rows, int l, int env_dtype, uint16_t *out, int rblocks, int kc, cudaStream_t st) {
    uimg_kernel<<<mt_grid((size_t)rblocks * kc * 1024), 256, 0, st>>>(U, rows, l, env_dtype, out, rblocks, kc);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}
mdbf_status_t launch_vimg(const void *V, int cols, int l, int env_dtype, uint16_t *out, int kblocks, int kc, cudaStream_t st) {
    vimg_kernel<<<mt_grid((size_t)kblocks * kc * 512), 256, 0, st>>>(V, cols, l, env_dtype, out, kblocks, kc);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

// 32 columns of one row of the A tile: envelope values -> bf16 pairs, sign bits XOR-ed in.
// `word` holds the row's 32 sign bits of these columns (bit set = -1); chunk c4 of 8 columns goes
// to the 16-byte slot (cbase + c4) ^ (row & 7) of the row (128B swizzle).
__device__ __forceinline__ void mt_expand_half(const uint32_t (&v)[32], uint32_t word, unsigned char *srow, int arow, int cbase) {
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) {
        const uint32_t byte = (word >> (8 * c4)) & 0xFFu;   // 8 bits: the two shifted copies in the product below cannot overlap
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int col = c4 * 8 + 2 * i;
            const uint32_t e = tm::pack_bf16x2(__uint_as_float(v[col]), __uint_as_float(v[col + 1]));
            // bit 0 of the shifted byte -> bit 15, bit 1 -> bit 31; the other product bits fall outside the mask
            const uint32_t m = ((byte >> (2 * i)) * 0x40008000u) & 0x80008000u;
            o[i] = e ^ m;
        }
        *reinterpret_cast<uint4 *>(srow + (((cbase + c4) ^ (arow & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

template <bool STAGE_A>
__global__ void __launch_bounds__(MT_THREADS, 1)
mat_stage_kernel(const MatArgs a, const __grid_constant__ CUtensorMap tmap_in) {
    using namespace tm;
    extern __shared__ unsigned char mt_smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * MT_MAX_NS + 2 * MT_NE + 2 * MT_MAX_NV + 2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(mt_smem_raw) + 1023u) & ~1023u;
    unsigned char *smem_gen = mt_smem_raw + (smem_base - smem_u32(mt_smem_raw));
    const int ns = a.ns, nv = a.nv;
    const uint32_t b_bytes = (uint32_t)a.bn * MT_BK * 2;
    const uint32_t stage_bytes = MT_A_BYTES + b_bytes;              // A tile, then the activation tile
    const uint32_t u_smem = smem_base + (uint32_t)ns * stage_bytes;
    const uint32_t u_bytes = (uint32_t)a.kc * 2048u, v_bytes = (uint32_t)a.kc * 1024u;
    const uint32_t v_smem = u_smem + u_bytes;                       // + vb * v_bytes
    const uint32_t full_bar = smem_u32(&bars[0]);
    const uint32_t empty_bar = full_bar + 8 * MT_MAX_NS;
    const uint32_t efull_bar = empty_bar + 8 * MT_MAX_NS;
    const uint32_t eempty_bar = efull_bar + 8 * MT_NE;
    const uint32_t vfull_bar = eempty_bar + 8 * MT_NE;
    const uint32_t vempty_bar = vfull_bar + 8 * MT_MAX_NV;
    const uint32_t accum_bar = vempty_bar + 8 * MT_MAX_NV;
    const uint32_t u_bar = accum_bar + 8;

    const int rb = blockIdx.x;
    const int row0 = rb * MT_BM;
    const int tau0 = blockIdx.y * a.bn;
    const int nkb = (a.cols + MT_BK - 1) / MT_BK;

    if (tid == 0) {
        for (int s = 0; s < MT_MAX_NS; ++s) {
            mbar_init(full_bar + 8 * s, 128 + 1);       // one expander group + the TMA issuer's expect_tx
            mbar_init(empty_bar + 8 * s, 1);
        }
        for (int e = 0; e < MT_NE; ++e) {
            mbar_init(efull_bar + 8 * e, 1);
            mbar_init(eempty_bar + 8 * e, 128);
        }
        for (int v = 0; v < MT_MAX_NV; ++v) {
            mbar_init(vfull_bar + 8 * v, 1);
            mbar_init(vempty_bar + 8 * v, 1);
        }
        mbar_init(accum_bar, 1);
        mbar_init(u_bar, 1);
        abort_flag_s = 0;
        fence_barrier_init();
    }
    if (warp == MT_W_MMA) {
        tmem_alloc(smem_u32(&tmem_base_slot), MT_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_slot;              // accumulator: columns 0 .. 255
    const uint32_t tmem_e = tmem_base_slot + MT_BN;      // envelope buffers: 64 columns each
    pdl_launch_dependents();

    if (warp < MT_W_TMA) {
        // ============================ W_hat tile builders ============================
        const int grp = warp >> 2;
        const int arow = tid & 127;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint2 *wp = a.wk + (size_t)row0 + arow;                       // + kb * rows_pad
        uint2 w_next = grp < nkb ? __ldg(wp + (size_t)grp * a.rows_pad) : make_uint2(0u, 0u);
        uint2 w_next2 = grp + MT_GROUPS < nkb ? __ldg(wp + (size_t)(grp + MT_GROUPS) * a.rows_pad) : make_uint2(0u, 0u);
        bool alive = true;
        int s = grp;                                      // ring slot and phase of K block kb (ns >= 4 > grp)
        uint32_t ph = 0;
        for (int kb = grp; kb < nkb && alive; kb += MT_GROUPS) {
            const int eb = kb & (MT_NE - 1);
            const uint32_t eph = (uint32_t)(kb / MT_NE) & 1u;
            const uint2 w = w_next;
            w_next = w_next2;
            if (kb + 2 * MT_GROUPS < nkb) w_next2 = __ldg(wp + (size_t)(kb + 2 * MT_GROUPS) * a.rows_pad);
            alive = mbar_wait(efull_bar + 8 * eb, eph, abort_flag, a.status);
            if (!alive) break;
            tc_fence_after();
            uint32_t v0[32], v1[32];
            tmem_ld32(tmem_e + (uint32_t)(eb * 64) + lane_base, v0);
            tmem_ld32(tmem_e + (uint32_t)(eb * 64 + 32) + lane_base, v1);
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(eempty_bar + 8 * eb);                                // the buffer may be overwritten
            alive = mbar_wait(empty_bar + 8 * s, ph ^ 1u, abort_flag, a.status);
            if (!alive) break;
            unsigned char *srow = smem_gen + (size_t)s * stage_bytes + arow * 128;
            mt_expand_half(v0, w.x, srow, arow, 0);
            mt_expand_half(v1, w.y, srow, arow, 4);
            fence_proxy_async();
            mbar_arrive(full_bar + 8 * s);
            s += MT_GROUPS;
            if (s >= ns) { s -= ns; ph ^= 1u; }
        }

        // ================================= epilogue ==================================
        const int egrow = row0 + arow;
        if (alive) alive = mbar_wait(accum_bar, 0u, abort_flag, a.status);
        tc_fence_after();
        pdl_wait();                                   // the stores below must follow the previous kernel's reads
        if (alive) {
#pragma unroll 1
            for (int ld = grp; ld * 32 < a.bn; ld += MT_GROUPS) {
                const int col0 = ld * 32;
                uint32_t v[32];
                tmem_ld32(tmem_d + lane_base + (uint32_t)col0, v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int tau = tau0 + col0 + j;
                    if (egrow < a.rows && col0 + j < a.bn && tau < a.T) {
                        const float acc = __uint_as_float(v[j]);
                        if (STAGE_A) {
                            if (a.y_mode == 0) a.y[(size_t)tau * a.rows + egrow] = __float2bfloat16_rn(acc);
                            else if (a.y_mode == 1) a.y32[(size_t)tau * a.rows + egrow] = acc;
                            else a.y32[(size_t)tau * a.rows + egrow] += acc;
                        } else {
                            a.zb[(size_t)tau * a.zstride + egrow] = __float2bfloat16_rn(acc);
                        }
                    }
                }
            }
        }
    } else if (warp == MT_W_TMA) {
        // ============================ activation-tile loader ===========================
        bool alive = true;
        pdl_wait();                                   // the activations come from the previous kernel
        int s = 0;
        uint32_t ph = 0;
        for (int kb = 0; kb < nkb && alive; ++kb) {
            alive = mbar_wait(empty_bar + 8 * s, ph ^ 1u, abort_flag, a.status);
            if (!alive) break;
            if (lane == 0) {
                mbar_arrive_expect_tx(full_bar + 8 * s, b_bytes);
                tma_load_2d(smem_base + (uint32_t)s * stage_bytes + MT_A_BYTES, &tmap_in, kb * MT_BK, tau0,
                            full_bar + 8 * s);
            }
            __syncwarp();
            if (++s == ns) { s = 0; ph ^= 1u; }
        }
        if (!alive) drain_delay();
    } else if (warp == MT_W_ENV) {
        // ============================= envelope-image loader ===========================
        bool alive = true;
        if (lane == 0) {
            mbar_arrive_expect_tx(u_bar, u_bytes);
            bulk_load(u_smem, a.uimg + (size_t)rb * (u_bytes / 2), u_bytes, u_bar);
        }
        int vb = 0;
        uint32_t vph = 0;
        for (int kb = 0; kb < nkb && alive; ++kb) {
            alive = mbar_wait(vempty_bar + 8 * vb, vph ^ 1u, abort_flag, a.status);
            if (!alive) break;
            if (lane == 0) {
                mbar_arrive_expect_tx(vfull_bar + 8 * vb, v_bytes);
                bulk_load(v_smem + (uint32_t)vb * v_bytes, a.vimg + (size_t)kb * (v_bytes / 2), v_bytes, vfull_bar + 8 * vb);
            }
            __syncwarp();
            if (++vb == nv) { vb = 0; vph ^= 1u; }
        }
        if (!alive) drain_delay();
    } else if (warp == MT_W_MINI) {
        // ===================== envelope mini-MMA issuer: E(j) = U image x V image(j)^T =====================
        // runs as far ahead of the main MMAs as the four TMEM buffers allow
        const uint32_t idesc_mini = make_idesc_fmt(MT_BK, a.env_fmt);
        bool alive = mbar_wait(u_bar, 0u, abort_flag, a.status);
        int vb = 0;
        uint32_t vph = 0;
        for (int j = 0; j < nkb && alive; ++j) {
            const int eb = j & (MT_NE - 1);
            alive = mbar_wait(vfull_bar + 8 * vb, vph, abort_flag, a.status);
            if (!alive) break;
            alive = mbar_wait(eempty_bar + 8 * eb, ((uint32_t)(j / MT_NE) & 1u) ^ 1u, abort_flag, a.status);
            if (!alive) break;
            tc_fence_after();
            if (lane == 0) {
                for (int q = 0; q < a.kc / 2; ++q) {
                    const uint64_t ud = make_smem_desc_plain(u_smem + (uint32_t)q * 4096u, 2048u, 128u);
                    const uint64_t vd = make_smem_desc_plain(v_smem + (uint32_t)vb * v_bytes + (uint32_t)q * 2048u, 1024u, 128u);
                    umma_ss(tmem_e + (uint32_t)(eb * 64), ud, vd, idesc_mini, q > 0 ? 1u : 0u);
                }
                umma_commit(efull_bar + 8 * eb);
                umma_commit(vempty_bar + 8 * vb);
            }
            __syncwarp();
            if (++vb == nv) { vb = 0; vph ^= 1u; }
        }
    } else {
        // ================================ main MMA issuer =================================
        const uint32_t idesc_main = make_idesc(a.bn);
        bool alive = true;
        int s = 0;
        uint32_t ph = 0;
        for (int kb = 0; kb < nkb && alive; ++kb) {
            alive = mbar_wait(full_bar + 8 * s, ph, abort_flag, a.status);
            if (!alive) break;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t sA = smem_base + (uint32_t)s * stage_bytes;
                const uint64_t adesc = make_smem_desc(sA);
                const uint64_t bdesc = make_smem_desc(sA + MT_A_BYTES);
#pragma unroll
                for (int k4 = 0; k4 < MT_BK / 16; ++k4)
                    umma_ss(tmem_d, adesc + (uint64_t)(2 * k4), bdesc + (uint64_t)(2 * k4), idesc_main,
                            (kb > 0 || k4 > 0) ? 1u : 0u);
                umma_commit(empty_bar + 8 * s);
            }
            __syncwarp();
            if (++s == ns) { s = 0; ph ^= 1u; }
        }
        if (lane == 0 && alive) { if (nkb > 0) umma_commit(accum_bar); else mbar_arrive(accum_bar); }
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == MT_W_MMA) tmem_dealloc(tmem_d, MT_TMEM_COLS);
}

// bf16 intermediate -> the fp32 inspection buffer
__global__ void zb_to_zsum_kernel(const __nv_bfloat16 *__restrict__ zb, int zstride, float *__restrict__ zsum, int T, int k) {
    const size_t total = (size_t)T * k;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int tau = (int)(idx / k), r = (int)(idx % k);
        zsum[idx] = __bfloat162float(zb[(size_t)tau * zstride + r]);
    }
}
mdbf_status_t launch_zb_to_zsum(Layer &L, int T, cudaStream_t st) {
    zb_to_zsum_kernel<<<mt_grid((size_t)T * L.d.k), 256, 0, st>>>(L.zb, L.padA, L.zsum, T, L.d.k);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

// The kernel reads x through a tensor map: 16-byte aligned base and row pitch.
bool mat_path_supports(const Layer &L, const void *x, int T) {
    return L.uiA && L.zb && T >= 2 && (reinterpret_cast<uintptr_t>(x) & 15u) == 0 && L.d.d_in % 8 == 0;
}

static int mt_ring(int bn) {
    const int n = MT_RING_BYTES / (MT_A_BYTES + bn * MT_BK * 2);
    return n < MT_MAX_NS ? n : MT_MAX_NS;
}
static size_t mt_smem_bytes(int kc, int nv, int bn) {
    return (size_t)mt_ring(bn) * (MT_A_BYTES + bn * MT_BK * 2) + (size_t)kc * 2048 + (size_t)nv * kc * 1024 + 1024;
}

template <bool STAGE_A>
static mdbf_status_t launch_mat(const MatArgs &a, const CUtensorMap &tm, cudaStream_t st) {
    static bool attr_set = false;
    if (!attr_set) {
        MDBF_CUDA(cudaFuncSetAttribute(mat_stage_kernel<STAGE_A>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)mt_smem_bytes(4, 6, MT_BN)));
        attr_set = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ceil_div(a.rows, MT_BM), ceil_div(a.T, a.bn), 1);
    cfg.blockDim = dim3(MT_THREADS);
    cfg.dynamicSmemBytes = mt_smem_bytes(a.kc, a.nv, a.bn);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    MDBF_CUDA(cudaLaunchKernelEx(&cfg, mat_stage_kernel<STAGE_A>, a, tm));
    return MDBF_OK;
}

mdbf_status_t launch_forward_mat(Layer &L, const void *x, void *y, int T, cudaStream_t st, int *launches) {
    const mdbf_desc_t &d = L.d;
    if (!mat_path_supports(L, x, T)) {
        set_error("mdbf_linear_forward: the materialised-envelope kernel needs T >= 2, max_T >= 2, 16-bit envelopes, "
                  "l <= 32, d_in a multiple of 8 and x aligned to 16 bytes");
        return MDBF_ERR_SHAPE;
    }
    const int bn = T >= MT_BN ? MT_BN : ((T + 15) / 16) * 16;
    CUtensorMap tmx, tmz;
    mdbf_status_t rc = make_act_tensor_map(&tmx, x, (size_t)T, d.d_in, d.d_in, bn);
    if (rc) return rc;
    rc = make_act_tensor_map(&tmz, L.zb, (size_t)T, d.k, L.padA, bn);
    if (rc) return rc;

    MatArgs b = {};
    b.wk = L.wkB; b.rows_pad = L.rpB; b.rows = d.k; b.cols = d.d_in;
    b.uimg = L.uiB; b.vimg = L.viB; b.kc = L.kcm; b.env_fmt = d.env_dtype == MDBF_BF16 ? 1u : 0u;
    b.nv = L.kcm == 2 ? 8 : 6;
    b.T = T; b.bn = bn; b.ns = mt_ring(bn); b.zb = L.zb; b.zstride = L.padA; b.status = L.status;
    rc = launch_mat<false>(b, tmx, st);
    if (rc) return rc;

    MatArgs a = {};
    a.wk = L.wkA; a.rows_pad = L.rpA; a.rows = d.d_out; a.cols = d.k;
    a.uimg = L.uiA; a.vimg = L.viA; a.kc = L.kcm; a.env_fmt = b.env_fmt; a.nv = b.nv;
    a.T = T; a.bn = bn; a.ns = b.ns;
    a.y = reinterpret_cast<__nv_bfloat16 *>(y); a.y32 = reinterpret_cast<float *>(y); a.y_mode = L.out_mode; a.status = L.status;
    rc = launch_mat<true>(a, tmz, st);
    if (rc) return rc;
    L.last_ksplit = -1;
    *launches = 2;
    return MDBF_OK;
}

}  // namespace mdbf
