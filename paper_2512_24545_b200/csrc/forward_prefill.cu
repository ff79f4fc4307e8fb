// Large-T ("prefill") path of the MDBF forward on the 5th-generation tensor
// cores: tcgen05.mma with the accumulator in tensor memory (TMEM).
//
// One stage is the dense contraction behind  sum_t D_{u_t} S D_{v_t}  (Eq.
// me-dbf-expand) over a block of tokens:
//
//     D[r][(tau, t)] = sum_c  S[r][c] * bf16( V[c][t] * in[tau][c] )        (GEMM, width l*T)
//     out[tau][r]    = sum_t  U[r][t] * D[r][(tau, t)]                      (fused epilogue)
//
// with A = S expanded to +-1.0 bf16 (M = 128 rows of S per CTA, K-major) and
// B = the envelope-scaled activations generated on the fly (N = 256 columns =
// 256/LP tokens x LP modes, K-major).  Stage B (S_B, V_B, U_B) maps x -> z,
// stage A (S_A, V_A, U_A) maps z -> y (Eq. DBF-inference-form).
//
// CTA = 9 warps.  Warps 0-7 are producers: per 64-column K block they expand
// the packed sign words into the 128B-swizzled A tile (a 16-entry nibble table
// turns 4 bits into four bf16 +-1) and write the B tile
// (fp32 multiply, one rounding to bf16), then publish the stage through an
// mbarrier after a generic->async proxy fence.  One lane of warp 8 issues the
// MMAs (4 x K=16 per stage) and commits each stage back to the producers; a
// 4-stage ring overlaps generation with the tensor pipe.  After the K loop the
// producer warps read the 128 x 256 fp32 accumulator from TMEM (tcgen05.ld),
// contract the LP modes of every token with U in registers and store.
//
// Every mbarrier wait is bounded: when it expires the kernel records
// MDBF_ERR_TIMEOUT in the layer's status word, all roles fall through to the
// common exit, TMEM is released and the kernel returns.
#include "common.cuh"

namespace mdbf {

constexpr int PF_BM = 128;
constexpr int PF_BN = 256;
constexpr int PF_BK = 64;
constexpr int PF_STAGES = 4;
constexpr int PF_PRODUCERS = 256;
constexpr int PF_THREADS = PF_PRODUCERS + 32;
constexpr int PF_A_BYTES = PF_BM * PF_BK * 2;      // 16 KB
constexpr int PF_B_BYTES = PF_BN * PF_BK * 2;      // 32 KB
constexpr int PF_STAGE_BYTES = PF_A_BYTES + PF_B_BYTES;
constexpr int PF_SMEM_BYTES = PF_STAGES * PF_STAGE_BYTES + 1024;   // + alignment slack
constexpr uint32_t PF_MAX_POLLS = 1u << 20;

struct PrefillArgs {
    const uint32_t *words;   // canonical sign words [rows][nwords]
    int nwords;
    int rows, cols;
    const void *U;           // [rows][l] env_dtype
    const uint16_t *Vp;      // private padded copy [cols_pad][LP], raw 16-bit env values, zero padded
    int env_dtype, l;
    const void *in;          // stage B: bf16 [T][cols]; stage A: fp32 [T][cols]
    void *out;               // stage B: fp32 [T][rows]; stage A: bf16 [T][rows]
    int T;
    int n_eff;               // MMA N: LP * tokens per tile actually used, multiple of 16
    int vec_ok;              // input rows are 16-byte aligned and cols % 8 == 0
    int32_t *status;
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait: false when it gave up (status word set, abort flag raised).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *status) {
    for (uint32_t it = 0; it < PF_MAX_POLLS; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(status, (int32_t)MDBF_ERR_TIMEOUT);
    return false;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }

// K-major operand tile with 128-byte rows and the 128B swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);          // start address
    d |= (uint64_t)1u << 16;                          // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)((1024u >> 4) & 0x3FFFu) << 32;    // stride byte offset between 8-row groups
    d |= (uint64_t)1u << 46;                          // descriptor version of this architecture
    d |= (uint64_t)2u << 61;                          // SWIZZLE_128B
    return d;
}
__device__ __forceinline__ uint32_t make_idesc(int n) {
    uint32_t d = 0;
    d |= 1u << 4;                       // D format: fp32
    d |= 1u << 7;                       // A format: bf16
    d |= 1u << 10;                      // B format: bf16
    d |= (uint32_t)(n >> 3) << 17;      // N
    d |= (uint32_t)(PF_BM >> 4) << 24;  // M
    return d;                           // A and B K-major, no negation, dense
}

__device__ __forceinline__ float raw16_to_float(uint16_t r, int dtype) {
    if (dtype == MDBF_F16) return __half2float(__ushort_as_half(r));
    return __uint_as_float((uint32_t)r << 16);
}
__device__ __forceinline__ uint32_t pf_pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// --------------------------------------------------------------------- kernel
template <int LP, bool STAGE_A>
__global__ void __launch_bounds__(PF_THREADS, 1) prefill_stage_kernel(const PrefillArgs a) {
    constexpr int TPT = LP < 4 ? LP : 4;        // modes per producer thread
    constexpr int TG = LP / TPT;                // mode groups
    constexpr int TAUPT = 8 / TPT;              // tokens per producer thread
    constexpr int TT = PF_BN / LP;              // tokens per CTA tile

    extern __shared__ unsigned char pf_smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * PF_STAGES + 1];
    __shared__ uint2 lut[16];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(pf_smem_raw) + 1023u) & ~1023u;
    unsigned char *smem_gen = pf_smem_raw + (smem_base - smem_u32(pf_smem_raw));
    const uint32_t full_bar = smem_u32(&bars[0]);                 // + 8*s
    const uint32_t empty_bar = smem_u32(&bars[PF_STAGES]);        // + 8*s
    const uint32_t accum_bar = smem_u32(&bars[2 * PF_STAGES]);

    const int row0 = blockIdx.x * PF_BM;
    const int tau0 = blockIdx.y * TT;
    const int nkb = (a.cols + PF_BK - 1) / PF_BK;

    if (tid == 0) {
        for (int s = 0; s < PF_STAGES; ++s) {
            mbar_init(full_bar + 8 * s, PF_PRODUCERS);
            mbar_init(empty_bar + 8 * s, 1);
        }
        mbar_init(accum_bar, 1);
        abort_flag_s = 0;
        fence_barrier_init();
    }
    if (tid < 16) {     // nibble -> four bf16 +-1.0 (bit set = -1), element i in half (i & 1) of word (i >> 1)
        uint32_t w0 = 0x3F803F80u, w1 = 0x3F803F80u;
        if (tid & 1) w0 |= 0x00008000u;
        if (tid & 2) w0 |= 0x80000000u;
        if (tid & 4) w1 |= 0x00008000u;
        if (tid & 8) w1 |= 0x80000000u;
        lut[tid] = make_uint2(w0, w1);
    }
    if (warp == 8) {
        tmem_alloc(smem_u32(&tmem_base_slot), PF_BN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_slot;

    if (warp < 8) {
        // ================================ producers ================================
        const int arow = tid & 127, ahalf = tid >> 7;                  // A: one 32-bit word per thread per stage
        const int grow = row0 + arow;
        const uint32_t *wrow = a.words + (size_t)(grow < a.rows ? grow : 0) * a.nwords;
        const bool arow_ok = grow < a.rows;
        const int kc = tid & 7;                                         // B: 16-byte chunk along K
        const int tg = (tid >> 3) % TG;
        const int taug = (tid >> 3) / TG;
        const int t_first = tg * TPT;

        auto load_word = [&](int kb) -> uint32_t {
            const int wi = kb * 2 + ahalf;
            return (arow_ok && wi < a.nwords) ? __ldg(wrow + wi) : 0u;
        };
        // raw prefetch registers for the next K block
        uint32_t aw_next = load_word(0);
        uint32_t vraw[8][(TPT + 1) / 2];       // 8 columns x TPT modes, 16-bit values packed in pairs
        float xin[TAUPT][8];
        auto load_v = [&](int kb) {
            const int c = kb * PF_BK + kc * 8;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint16_t *p = a.Vp + (size_t)(c + i) * LP + t_first;
                if (TPT == 4) { const uint2 v = __ldg(reinterpret_cast<const uint2 *>(p)); vraw[i][0] = v.x; vraw[i][1] = v.y; }
                else if (TPT == 2) vraw[i][0] = __ldg(reinterpret_cast<const uint32_t *>(p));
                else vraw[i][0] = __ldg(p);
            }
        };
        auto load_x = [&](int kb) {
            const int c = kb * PF_BK + kc * 8;
#pragma unroll
            for (int j = 0; j < TAUPT; ++j) {
                const int tau = tau0 + taug * TAUPT + j;
                if (tau < a.T && a.vec_ok && c + 8 <= a.cols) {
                    if (STAGE_A) {
                        const float4 *p = reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(a.in) + (size_t)tau * a.cols + c);
                        const float4 lo = __ldg(p), hi = __ldg(p + 1);
                        xin[j][0] = lo.x; xin[j][1] = lo.y; xin[j][2] = lo.z; xin[j][3] = lo.w;
                        xin[j][4] = hi.x; xin[j][5] = hi.y; xin[j][6] = hi.z; xin[j][7] = hi.w;
                    } else {
                        const uint4 r = __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(a.in) + (size_t)tau * a.cols + c));
                        const uint32_t rr[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            xin[j][2 * e] = __uint_as_float(rr[e] << 16);
                            xin[j][2 * e + 1] = __uint_as_float(rr[e] & 0xFFFF0000u);
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float v = 0.f;
                        if (tau < a.T && c + i < a.cols) {
                            if (STAGE_A) v = reinterpret_cast<const float *>(a.in)[(size_t)tau * a.cols + c + i];
                            else v = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(a.in)[(size_t)tau * a.cols + c + i]);
                        }
                        xin[j][i] = v;
                    }
                }
            }
        };
        load_v(0);
        load_x(0);

        bool alive = true;
        for (int kb = 0; kb < nkb && alive; ++kb) {
            const int s = kb % PF_STAGES;
            const uint32_t ph = (uint32_t)(kb / PF_STAGES) & 1u;
            // consume the prefetched registers
            const uint32_t aw = aw_next;
            float vf[8][TPT];
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int tt = 0; tt < TPT; ++tt) {
                    const uint32_t pr = vraw[i][tt >> 1];
                    vf[i][tt] = raw16_to_float((uint16_t)((tt & 1) ? (pr >> 16) : (pr & 0xFFFFu)), a.env_dtype);
                }
            float xf[TAUPT][8];
#pragma unroll
            for (int j = 0; j < TAUPT; ++j)
#pragma unroll
                for (int i = 0; i < 8; ++i) xf[j][i] = xin[j][i];
            if (kb + 1 < nkb) { aw_next = load_word(kb + 1); load_v(kb + 1); load_x(kb + 1); }

            alive = mbar_wait(empty_bar + 8 * s, ph ^ 1u, abort_flag, a.status);
            if (!alive) break;
            unsigned char *sA = smem_gen + (size_t)s * PF_STAGE_BYTES;
            unsigned char *sB = sA + PF_A_BYTES;
            // A: 32 bits -> four 16-byte chunks of row `arow`
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t byte = (aw >> (8 * j)) & 0xFFu;
                const uint2 lo = lut[byte & 15u], hi = lut[byte >> 4];
                const int c8 = ahalf * 4 + j;
                *reinterpret_cast<uint4 *>(sA + arow * 128 + ((c8 ^ (arow & 7)) << 4)) = make_uint4(lo.x, lo.y, hi.x, hi.y);
            }
            // B: rows n = tau_local * LP + t, chunk kc
#pragma unroll
            for (int j = 0; j < TAUPT; ++j) {
                const int taul = taug * TAUPT + j;
#pragma unroll
                for (int tt = 0; tt < TPT; ++tt) {
                    const int n = taul * LP + t_first + tt;
                    uint4 o;
                    o.x = pf_pack_bf16x2(vf[0][tt] * xf[j][0], vf[1][tt] * xf[j][1]);
                    o.y = pf_pack_bf16x2(vf[2][tt] * xf[j][2], vf[3][tt] * xf[j][3]);
                    o.z = pf_pack_bf16x2(vf[4][tt] * xf[j][4], vf[5][tt] * xf[j][5]);
                    o.w = pf_pack_bf16x2(vf[6][tt] * xf[j][6], vf[7][tt] * xf[j][7]);
                    if (n < a.n_eff)
                        *reinterpret_cast<uint4 *>(sB + n * 128 + ((kc ^ (n & 7)) << 4)) = o;
                }
            }
            fence_proxy_async();
            mbar_arrive(full_bar + 8 * s);
        }

        // ================================ epilogue =================================
        // warp w reads TMEM lanes 32*(w & 3) .. +31 (= rows of the tile), columns 128*(w >> 2) .. +127
        const int erow = (warp & 3) * 32 + lane;
        const int egrow = row0 + erow;
        const int chalf = warp >> 2;
        float u[LP];
#pragma unroll
        for (int t = 0; t < LP; ++t)
            u[t] = (egrow < a.rows && t < a.l) ? env_load(a.U, (size_t)egrow * a.l + t, a.env_dtype) : 0.f;
        if (alive) alive = mbar_wait(accum_bar, 0u, abort_flag, a.status);
        tc_fence_after();
        if (alive) {
            float acc = 0.f;
#pragma unroll
            for (int ld = 0; ld < 4; ++ld) {
                const int col0 = chalf * 128 + ld * 32;
                if (col0 < a.n_eff) {                                   // warp-uniform
                    uint32_t v[32];
                    tmem_ld32(tmem_d + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)col0, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int n = col0 + j;
                        const int t = n % LP;
                        acc += u[t] * __uint_as_float(v[j]);
                        if (t == LP - 1) {
                            const int tau = tau0 + n / LP;
                            if (egrow < a.rows && tau < a.T) {
                                if (STAGE_A) reinterpret_cast<__nv_bfloat16 *>(a.out)[(size_t)tau * a.rows + egrow] = __float2bfloat16_rn(acc);
                                else reinterpret_cast<float *>(a.out)[(size_t)tau * a.rows + egrow] = acc;
                            }
                            acc = 0.f;
                        }
                    }
                }
            }
        }
    } else {
        // ================================ MMA issuer ===============================
        const uint32_t idesc = make_idesc(a.n_eff);
        bool alive = true;
        for (int kb = 0; kb < nkb && alive; ++kb) {
            const int s = kb % PF_STAGES;
            const uint32_t ph = (uint32_t)(kb / PF_STAGES) & 1u;
            alive = mbar_wait(full_bar + 8 * s, ph, abort_flag, a.status);
            if (!alive) break;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t sA = smem_base + (uint32_t)s * PF_STAGE_BYTES;
                const uint64_t adesc = make_smem_desc(sA);
                const uint64_t bdesc = make_smem_desc(sA + PF_A_BYTES);
#pragma unroll
                for (int k4 = 0; k4 < PF_BK / 16; ++k4)
                    umma_bf16(tmem_d, adesc + (uint64_t)(2 * k4), bdesc + (uint64_t)(2 * k4), idesc,
                              (kb > 0 || k4 > 0) ? 1u : 0u);
                umma_commit(empty_bar + 8 * s);       // stage reusable once these MMAs retire
            }
            __syncwarp();
        }
        if (lane == 0 && alive) umma_commit(accum_bar);
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem_d, PF_BN);
}

// private padded copy of V: [cols_pad][LP] raw 16-bit values of the stored envelope type
__global__ void vpad_kernel(const void *__restrict__ V, int cols, int l, int env_dtype, uint16_t *__restrict__ out,
                            int cols_pad, int LP) {
    const size_t total = (size_t)cols_pad * LP;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(idx / LP), t = (int)(idx % LP);
        uint16_t r = 0;
        if (c < cols && t < l) r = reinterpret_cast<const uint16_t *>(V)[(size_t)c * l + t];
        out[idx] = r;
    }
}

mdbf_status_t launch_vpad(const void *V, int cols, int l, int env_dtype, uint16_t *out, int cols_pad, int LP,
                          cudaStream_t st) {
    const size_t total = (size_t)cols_pad * LP;
    int grid = (int)((total + 255) / 256);
    if (grid > 148 * 16) grid = 148 * 16;
    vpad_kernel<<<grid, 256, 0, st>>>(V, cols, l, env_dtype, out, cols_pad, LP);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

template <int LP, bool STAGE_A>
static mdbf_status_t launch_pf(const PrefillArgs &a, cudaStream_t st) {
    auto kern = prefill_stage_kernel<LP, STAGE_A>;
    static bool attr_set = false;
    if (!attr_set) {
        MDBF_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, PF_SMEM_BYTES));
        attr_set = true;
    }
    const int TT = PF_BN / LP;
    dim3 grid(ceil_div(a.rows, PF_BM), ceil_div(a.T, TT));
    kern<<<grid, PF_THREADS, PF_SMEM_BYTES, st>>>(a);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

template <bool STAGE_A>
static mdbf_status_t dispatch_pf(int LP, const PrefillArgs &a, cudaStream_t st) {
    switch (LP) {
        case 1: return launch_pf<1, STAGE_A>(a, st);
        case 2: return launch_pf<2, STAGE_A>(a, st);
        case 4: return launch_pf<4, STAGE_A>(a, st);
        case 8: return launch_pf<8, STAGE_A>(a, st);
        case 16: return launch_pf<16, STAGE_A>(a, st);
        case 32: return launch_pf<32, STAGE_A>(a, st);
        case 64: return launch_pf<64, STAGE_A>(a, st);
    }
    set_error("prefill stage: unsupported padded envelope rank %d", LP);
    return MDBF_ERR_SHAPE;
}

mdbf_status_t launch_forward_prefill(Layer &L, const void *x, void *y, int T, cudaStream_t st, int *launches) {
    const mdbf_desc_t &d = L.d;
    const int LP = L.LP;
    const int TT = PF_BN / LP;
    const int tok = T < TT ? T : TT;
    const int n_eff = ((tok * LP + 15) / 16) * 16;
    PrefillArgs b = {};
    b.words = L.wB; b.nwords = L.wordsB; b.rows = d.k; b.cols = d.d_in;
    b.U = L.UB; b.Vp = L.vpB; b.env_dtype = d.env_dtype; b.l = d.l;
    b.in = x; b.out = L.zsum; b.T = T; b.n_eff = n_eff;
    b.vec_ok = ((reinterpret_cast<uintptr_t>(x) & 15u) == 0 && d.d_in % 8 == 0) ? 1 : 0;
    b.status = L.status;
    mdbf_status_t rc = dispatch_pf<false>(LP, b, st);
    if (rc) return rc;
    PrefillArgs a = {};
    a.words = L.wA; a.nwords = L.wordsA; a.rows = d.d_out; a.cols = d.k;
    a.U = L.UA; a.Vp = L.vpA; a.env_dtype = d.env_dtype; a.l = d.l;
    a.in = L.zsum; a.out = y; a.T = T; a.n_eff = n_eff;
    a.vec_ok = (d.k % 8 == 0) ? 1 : 0;
    a.status = L.status;
    rc = dispatch_pf<true>(LP, a, st);
    if (rc) return rc;
    L.last_ksplit = 0;
    *launches = 2;
    return MDBF_OK;
}

}  // namespace mdbf
