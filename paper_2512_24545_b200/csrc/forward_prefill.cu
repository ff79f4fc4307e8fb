// Large-T ("prefill") path of the MDBF forward on the 5th-generation tensor
// cores: tcgen05.mma with the accumulator in tensor memory (TMEM), the
// activation operand staged by TMA, the sign operand expanded in shared memory.
//
// One stage is the dense contraction behind  sum_t D_{u_t} S D_{v_t}  (Eq.
// me-dbf-expand) over a block of tokens:
//
//     Xs[(tau, t)][c] = bf16( V[c][t] * in[tau][c] )                        (pre-scale, one rounding)
//     D[r][(tau, t)]  = sum_c  S[r][c] * Xs[(tau, t)][c]                    (GEMM, width l*T, fp32 acc)
//     out[tau][r]     = sum_t  U[r][t] * D[r][(tau, t)]                     (fused epilogue)
//
// Stage B (S_B, V_B, U_B) maps x -> z, stage A (S_A, V_A, U_A) maps z -> y
// (Eq. DBF-inference-form, column convention).  Three launches per forward:
//
//   prescale_kernel      Xs_B from x and V_B (element-wise, HBM-bound, ~l*T*d_in*2 bytes written)
//   gemm_stage_kernel<B> z, and in the same epilogue Xs_A = bf16(V_A * z) for the next stage
//   gemm_stage_kernel<A> y
//
// GEMM CTA = 128 rows of S x 256 columns (256/LP tokens x LP modes), 10 warps:
//   warps 0-7  two groups of four; group g expands, for the K blocks g, g+2, ..., 64 packed sign
//              bits per row into the 128B-swizzled bf16 A tile (+-1.0; three integer ops per pair
//              of elements); later both groups run the epilogue on alternate 32-column chunks
//   warp 8     one lane issues the TMA load of the Xs tile (tensor map, 128B swizzle; box of 64,
//              128 or 256 rows)
//   warp 9     one lane issues 4 tcgen05.mma (K = 16 each) per K block and commits the stage
// in a 4-stage mbarrier ring.  The epilogue reads the 128 x 256 fp32 accumulator from TMEM
// (tcgen05.ld), contracts the LP modes of every token with U in registers and stores.
//
// Generating Xs on the fly inside the GEMM was measured first and rejected: the per-stage
// global loads and 16-bit conversions saturated the load/store and conversion pipes
// (tensor pipe 18 % busy); the pre-scaled operand costs < 10 % extra HBM time and removes
// all of it.
//
// Every mbarrier wait is bounded: when it expires the kernel records MDBF_ERR_TIMEOUT in
// the layer's status word, all roles fall through to the common exit, TMEM is released and
// the kernel returns.  Every TMA and bulk copy targets the issuing CTA's own shared memory only.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace mdbf {

constexpr int PF_BM = 128;
constexpr int PF_BN = 256;
constexpr int PF_BK = 64;
constexpr int PF_STAGES = 4;
constexpr int PF_EXPANDERS = 128;                  // threads that fill one A tile (one per row)
constexpr int PF_GROUPS = 2;                       // expander groups: group g fills the tiles of K blocks g, g + 2, ...
constexpr int PF_W_TMA = PF_GROUPS * 4;            // warp indices of the two single-lane roles
constexpr int PF_W_MMA = PF_W_TMA + 1;
constexpr int PF_THREADS = PF_GROUPS * PF_EXPANDERS + 64;
constexpr int PF_A_BYTES = PF_BM * PF_BK * 2;      // 16 KB
constexpr int PF_B_BYTES = PF_BN * PF_BK * 2;      // 32 KB
constexpr int PF_STAGE_BYTES = PF_A_BYTES + PF_B_BYTES;
constexpr int PF_PART_BYTES = 32 * 1024;           // partial outputs pushed by the ranks of a split cluster: [rank][token][128] fp32
constexpr int PF_SMEM_BYTES = PF_STAGES * PF_STAGE_BYTES + PF_PART_BYTES + 1024;   // + alignment slack
constexpr uint32_t PF_MAX_POLLS = 1u << 20;

struct GemmArgs {
    const uint2 *wk;         // K-blocked sign words [kblocks][rows_pad], 64 bits per row and block
    int rows_pad;
    int rows, cols;
    const void *U;           // [rows][l] env_dtype
    int env_dtype, l;
    int T;
    int n_eff;               // MMA N: columns of the tile actually used, multiple of 16
    // stage B only: z out and the next stage's pre-scaled operand
    float *z;                // [T][rows] fp32
    const void *Vnext;       // V_A [rows][l] env_dtype
    __nv_bfloat16 *xs_next;  // [(tau, t)][pad_next]
    int pad_next;
    // stage A only
    __nv_bfloat16 *y;        // [T][rows]
    float *y32;              // [T][rows]: fp32 output when the layer is a term of a sum (y_mode 1: store, 2: add)
    int y_mode;
    int box_rows;            // rows of the TMA box of the Xs operand: 64, 128 or 256 (>= n_eff)
    int kb_per_cta;          // K blocks per cluster rank (blockIdx.z); the ranks' partial outputs are reduced over DSMEM
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
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
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
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }
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
// 2-D tiled TMA load into this CTA's shared memory, completion on an mbarrier (one destination CTA).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tmap, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(bar) : "memory");
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

__device__ __forceinline__ uint32_t pf_pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
// bits (2i, 2i+1) of an 8-bit value -> two bf16 +-1.0 (bit set = -1.0): the multiply moves bit 0
// to position 15 and bit 1 to position 31; every other product bit falls outside the mask.
__device__ __forceinline__ uint32_t sign_pair(uint32_t byte, int i) {
    return (((byte >> (2 * i)) * 0x40008000u) & 0x80008000u) | 0x3F803F80u;
}

// ----------------------------------------------------------------- GEMM stage
template <int LP, bool STAGE_A, bool SPLIT>
__global__ void __launch_bounds__(PF_THREADS, 1)
gemm_stage_kernel(const GemmArgs a, const __grid_constant__ CUtensorMap tmap_xs) {
    constexpr int TT = PF_BN / LP;              // tokens per CTA tile

    extern __shared__ unsigned char pf_smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * PF_STAGES + 1];
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
    const int nkb_total = (a.cols + PF_BK - 1) / PF_BK;
    const int kb0 = SPLIT ? blockIdx.z * a.kb_per_cta : 0;   // this cluster rank's slice of the reduction
    const int nkb = SPLIT ? max(0, min(a.kb_per_cta, nkb_total - kb0)) : nkb_total;
    constexpr bool split = SPLIT;                            // the reduction is shared by the ranks of a cluster
    cg::cluster_group cluster = cg::this_cluster();

    if (tid == 0) {
        for (int s = 0; s < PF_STAGES; ++s) {
            mbar_init(full_bar + 8 * s, PF_EXPANDERS + 1);   // expander threads + the TMA issuer's expect_tx
            mbar_init(empty_bar + 8 * s, 1);
        }
        mbar_init(accum_bar, 1);
        abort_flag_s = 0;
        fence_barrier_init();
    }
    if (warp == PF_W_MMA) {
        tmem_alloc(smem_u32(&tmem_base_slot), PF_BN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_slot;
    // Programmatic dependent launch: the next kernel may start its prologue now; whatever reads or
    // overwrites data of the previous kernel (the Xs operand, z / Xs_next / y) waits for it below.
    pdl_launch_dependents();

    if (warp < PF_W_TMA) {
        // ============================ sign-tile expanders ============================
        // Two groups of four warps work on alternate K blocks: one warp's walk through a block is a
        // chain of fixed latencies (barrier test, loads, shared stores, fence), so two blocks in
        // flight nearly double the rate at which tiles reach the tensor core.
        const int grp = warp >> 2;
        const int arow = tid & (PF_EXPANDERS - 1);                // one row of the tile per thread
        const uint2 *wp = a.wk + (size_t)kb0 * a.rows_pad + (size_t)row0 + arow;   // + kb * rows_pad
        uint2 w_next = grp < nkb ? __ldg(wp + (size_t)grp * a.rows_pad) : make_uint2(0u, 0u);
        bool alive = true;
        for (int kb = grp; kb < nkb && alive; kb += PF_GROUPS) {
            const int s = kb % PF_STAGES;
            const uint32_t ph = (uint32_t)(kb / PF_STAGES) & 1u;
            const uint2 w = w_next;
            if (kb + PF_GROUPS < nkb) w_next = __ldg(wp + (size_t)(kb + PF_GROUPS) * a.rows_pad);
            alive = mbar_wait(empty_bar + 8 * s, ph ^ 1u, abort_flag, a.status);
            if (!alive) break;
            unsigned char *sA = smem_gen + (size_t)s * PF_STAGE_BYTES + arow * 128;
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) {                      // 8 columns -> one 16-byte chunk
                const uint32_t byte = ((c8 < 4 ? w.x : w.y) >> (8 * (c8 & 3))) & 0xFFu;
                *reinterpret_cast<uint4 *>(sA + ((c8 ^ (arow & 7)) << 4)) =
                    make_uint4(sign_pair(byte, 0), sign_pair(byte, 1), sign_pair(byte, 2), sign_pair(byte, 3));
            }
            fence_proxy_async();
            mbar_arrive(full_bar + 8 * s);
        }

        // ================================= epilogue ==================================
        // thread = TMEM lane = row of the tile; columns n = tau_local * LP + t
        const int egrow = row0 + arow;
        float u[LP], vn[STAGE_A ? 1 : LP];
#pragma unroll
        for (int t = 0; t < LP; ++t) {
            const bool ok = egrow < a.rows && t < a.l;
            u[t] = ok ? env_load(a.U, (size_t)egrow * a.l + t, a.env_dtype) : 0.f;
            if (!STAGE_A) vn[t] = ok ? env_load(a.Vnext, (size_t)egrow * a.l + t, a.env_dtype) : 0.f;
        }
        if (alive) alive = mbar_wait(accum_bar, 0u, abort_flag, a.status);
        tc_fence_after();
        pdl_wait();                                   // the stores below must follow the previous kernel's reads
        // one finished output value: stored at once, or parked for the cluster reduction
        // [rank][token of the tile][128 rows], a region of its own: other ranks write into it while this
        // CTA's pipeline stages may still be busy
        float *part = reinterpret_cast<float *>(smem_gen + PF_STAGES * PF_STAGE_BYTES);
        const unsigned crank = SPLIT ? cluster.block_rank() : 0u;
        const int ntl = ((a.n_eff + 31) / 32 * 32) / LP;      // token slots the read-out loop below produces (32 columns at a time)
        float *part_dst = SPLIT ? cluster.map_shared_rank(part, 0) : part;
        auto emit = [&](int tau, float acc) {
            if (egrow < a.rows && tau < a.T) {
                const size_t o = (size_t)tau * a.rows + egrow;
                if (!store_in_bounds(o, (size_t)a.T * a.rows, a.status)) return;
                if (STAGE_A) {
                    if (a.y_mode == 0) a.y[o] = __float2bfloat16_rn(acc);
                    else if (a.y_mode == 1) a.y32[o] = acc;
                    else a.y32[o] += acc;
                } else {
                    a.z[o] = acc;
                    // pre-scaled operand of stage A: [(tau, mode)][pad_next] entries, this row's column
                    if (!store_in_bounds((size_t)(tau * LP + LP - 1) * a.pad_next + egrow, (size_t)a.T * LP * a.pad_next, a.status)) return;
                    __nv_bfloat16 *xo = a.xs_next + (size_t)tau * LP * a.pad_next + egrow;
#pragma unroll
                    for (int t2 = 0; t2 < LP; ++t2)
                        xo[(size_t)t2 * a.pad_next] = __float2bfloat16_rn(vn[t2] * acc);
                }
            }
        };
        if (alive) {
            float acc = 0.f;
#pragma unroll 1
            for (int ld = grp; ld < PF_BN / 32; ld += PF_GROUPS) {      // the groups share a lane quadrant: alternate chunks
                const int col0 = ld * 32;
                if (col0 >= a.n_eff) break;                              // warp-uniform
                uint32_t v[32];
                if (!SPLIT || nkb > 0) {
                    tmem_ld32(tmem_d + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)col0, v);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;              // an empty slice contributes nothing
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int t = j % LP;                // col0 is a multiple of 32 and LP divides 32
                    acc += u[t] * __uint_as_float(v[j]);
                    if (t == LP - 1) {
                        const int tl = (col0 + j) / LP;
                        if (split) part_dst[((int)crank * ntl + tl) * PF_BM + arow] = acc;
                        else emit(tau0 + tl, acc);
                        acc = 0.f;
                    }
                }
            }
        }
        if (split) {
            // every rank has pushed its partial sums into rank 0's shared memory ([rank][token][row]);
            // after one cluster barrier rank 0 adds them up in rank order (deterministic) and stores
            tc_fence_before();
            cluster.sync();
            if (crank == 0 && alive && !*abort_flag) {
                const unsigned nranks = cluster.num_blocks();
                for (int tl = grp; tl < ntl; tl += PF_GROUPS) {
                    float acc = 0.f;
                    for (unsigned rk = 0; rk < nranks; ++rk) acc += part[((int)rk * ntl + tl) * PF_BM + arow];
                    emit(tau0 + tl, acc);
                }
            }
        }
    } else if (warp == PF_W_TMA) {
        // ================================ TMA issuer =================================
        bool alive = true;
        pdl_wait();                                   // Xs comes from the previous kernel
        for (int kb = 0; kb < nkb && alive; ++kb) {
            const int s = kb % PF_STAGES;
            const uint32_t ph = (uint32_t)(kb / PF_STAGES) & 1u;
            alive = mbar_wait(empty_bar + 8 * s, ph ^ 1u, abort_flag, a.status);
            if (!alive) break;
            if (lane == 0) {
                mbar_arrive_expect_tx(full_bar + 8 * s, (uint32_t)a.box_rows * PF_BK * 2);
                tma_load_2d(smem_base + (uint32_t)s * PF_STAGE_BYTES + PF_A_BYTES, &tmap_xs,
                            (kb0 + kb) * PF_BK, tau0 * LP, full_bar + 8 * s);
            }
            __syncwarp();
        }
    } else {
        // ================================ MMA issuer =================================
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
        if (lane == 0 && alive) { if (nkb > 0) umma_commit(accum_bar); else mbar_arrive(accum_bar); }
        __syncwarp();
    }
    if (split && warp >= PF_W_TMA) cluster.sync();          // the expander warps run this barrier inside their epilogue

    tc_fence_before();
    __syncthreads();
    if (warp == PF_W_MMA) tmem_dealloc(tmem_d, PF_BN);
}

// ------------------------------------------------------------------- pre-scale
// Xs[(tau*LP + t) * pad + c] = bf16( Vt[t][c] * x[tau][c] ), zero for c >= cols.
// One thread per (tau, 8 columns) and, with TS > 1 (few tokens: more threads to cover the load
// latency), per mode: thread handles LP / TS modes.
template <int LP, int TS>
__global__ void __launch_bounds__(256)
prescale_kernel(const __nv_bfloat16 *__restrict__ x, const float *__restrict__ Vt, __nv_bfloat16 *__restrict__ xs,
                int T, int cols, int pad, int vec_ok) {
    const int chunks = pad / 8;
    constexpr int MODES = LP / TS;
    const size_t total = (size_t)T * chunks * TS;
    pdl_launch_dependents();
    pdl_wait();                                       // x may come from, and Xs may still be read by, earlier kernels
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(idx % chunks) * 8;
        const int tg = (int)((idx / chunks) % TS), tau = (int)(idx / ((size_t)chunks * TS));
        float xv[8];
        if (vec_ok && c + 8 <= cols) {
            const uint4 r = __ldg(reinterpret_cast<const uint4 *>(x + (size_t)tau * cols + c));
            const uint32_t rr[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                xv[2 * e] = __uint_as_float(rr[e] << 16);
                xv[2 * e + 1] = __uint_as_float(rr[e] & 0xFFFF0000u);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) xv[i] = (c + i < cols) ? __bfloat162float(x[(size_t)tau * cols + c + i]) : 0.f;
        }
#pragma unroll
        for (int tm = 0; tm < MODES; ++tm) {
            const int t = tg * MODES + tm;
            const float4 v0 = __ldg(reinterpret_cast<const float4 *>(Vt + (size_t)t * pad + c));
            const float4 v1 = __ldg(reinterpret_cast<const float4 *>(Vt + (size_t)t * pad + c + 4));
            uint4 o;
            o.x = pf_pack_bf16x2(v0.x * xv[0], v0.y * xv[1]);
            o.y = pf_pack_bf16x2(v0.z * xv[2], v0.w * xv[3]);
            o.z = pf_pack_bf16x2(v1.x * xv[4], v1.y * xv[5]);
            o.w = pf_pack_bf16x2(v1.z * xv[6], v1.w * xv[7]);
            *reinterpret_cast<uint4 *>(xs + ((size_t)tau * LP + t) * pad + c) = o;
        }
    }
}

// --------------------------------------------------------- pack-time private copies
// K-blocked sign words: out[kb * rows_pad + r] = words (2kb, 2kb+1) of row r, zero outside the matrix.
__global__ void kblock_kernel(const SignView sv, int rows, uint2 *__restrict__ out, int rows_pad, int kblocks) {
    const int nwords = sv.nwords;
    const size_t total = (size_t)kblocks * rows_pad;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int kb = (int)(idx / rows_pad), r = (int)(idx % rows_pad);
        uint2 v = make_uint2(0u, 0u);
        if (r < rows) {
            if (2 * kb < nwords) v.x = sv.word(r, 2 * kb);
            if (2 * kb + 1 < nwords) v.y = sv.word(r, 2 * kb + 1);
        }
        out[idx] = v;
    }
}
// transposed fp32 copy of V: out[t * pad + c] = V[c][t], zero outside
__global__ void vtrans_kernel(const void *__restrict__ V, int cols, int l, int env_dtype, float *__restrict__ out,
                              int pad, int LP) {
    const size_t total = (size_t)LP * pad;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int t = (int)(idx / pad), c = (int)(idx % pad);
        out[idx] = (c < cols && t < l) ? env_load(V, (size_t)c * l + t, env_dtype) : 0.f;
    }
}

static int pf_grid(size_t items) {
    size_t g = (items + 255) / 256;
    if (g < 1) g = 1;
    if (g > 148 * 32) g = 148 * 32;
    return (int)g;
}

mdbf_status_t launch_kblock(const SignView &sv, int rows, uint2 *out, int rows_pad, int kblocks, cudaStream_t st) {
    kblock_kernel<<<pf_grid((size_t)kblocks * rows_pad), 256, 0, st>>>(sv, rows, out, rows_pad, kblocks);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}
// canonical words of a sign matrix from whichever copy the layer keeps (mdbf_get_packed)
__global__ void canon_kernel(const SignView sv, int rows, uint32_t *__restrict__ out) {
    const size_t total = (size_t)rows * sv.nwords;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x)
        out[idx] = sv.word((int)(idx / sv.nwords), (int)(idx % sv.nwords));
}
mdbf_status_t launch_canon(const SignView &sv, int rows, uint32_t *out, cudaStream_t st) {
    canon_kernel<<<pf_grid((size_t)rows * sv.nwords), 256, 0, st>>>(sv, rows, out);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}
mdbf_status_t launch_vtrans(const void *V, int cols, int l, int env_dtype, float *out, int pad, int LP, cudaStream_t st) {
    vtrans_kernel<<<pf_grid((size_t)LP * pad), 256, 0, st>>>(V, cols, l, env_dtype, out, pad, LP);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

// Tensor map of a bf16 activation matrix [rows][cols] whose rows are `stride` elements apart: box of 64
// columns x box_rows rows, 128B swizzle, zero fill outside the matrix.
mdbf_status_t make_act_tensor_map(CUtensorMap *out, const void *base, size_t rows, int cols, int stride, int box_rows) {
    typedef CUresult (*encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static encode_fn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        MDBF_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q));
        if (!p || q != cudaDriverEntryPointSuccess) {
            set_error("cuTensorMapEncodeTiled is not available from the driver");
            return MDBF_ERR_CUDA;
        }
        fn = reinterpret_cast<encode_fn>(p);
    }
    const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)stride * 2};
    const cuuint32_t box[2] = {PF_BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return MDBF_ERR_CUDA;
    }
    return MDBF_OK;
}
// Tensor map of a pre-scaled operand: bf16 [rows][pad] row-major.
mdbf_status_t make_xs_tensor_map(CUtensorMap *out, const void *base, size_t rows, int pad, int box_rows) {
    return make_act_tensor_map(out, base, rows, pad, pad, box_rows);
}

// ---------------------------------------------------------------------- launch
template <int LP, bool STAGE_A>
static mdbf_status_t launch_gemm(const GemmArgs &a, const CUtensorMap &tm, cudaStream_t st) {
    static PerDeviceOnce once;
    if (once.first()) {
        MDBF_CUDA(cudaFuncSetAttribute(gemm_stage_kernel<LP, STAGE_A, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PF_SMEM_BYTES));
        MDBF_CUDA(cudaFuncSetAttribute(gemm_stage_kernel<LP, STAGE_A, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PF_SMEM_BYTES));
    }
    const int TT = PF_BN / LP;
    const int rb = ceil_div(a.rows, PF_BM), ntiles = ceil_div(a.T, TT), nkb = ceil_div(a.cols, PF_BK);
    // Few tokens leave most SMs without a tile: split the reduction over a cluster of up to 8 CTAs
    // (partial outputs reduced through DSMEM).  Cost model: waves x (K blocks per CTA + fixed part).
    int best_ks = 1;
    long best_cost = -1;
    for (int ks = 1; ks <= 8; ks *= 2) {
        const int per = ceil_div(nkb, ks);
        if (ks > 1 && per * (ks - 1) >= nkb) continue;                 // an empty rank
        if (ks > 1 && (size_t)ks * (((a.n_eff + 31) / 32 * 32) / LP) * PF_BM * sizeof(float) > PF_PART_BYTES) continue;   // partials must fit
        const long waves = ceil_div((long)rb * ntiles * ks, 148);
        const long cost = waves * (per + 10);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_ks = ks; }
    }
    GemmArgs args = a;
    args.kb_per_cta = ceil_div(nkb, best_ks);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(rb, ntiles, best_ks);
    cfg.blockDim = dim3(PF_THREADS);
    cfg.dynamicSmemBytes = PF_SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = best_ks;
    cfg.attrs = attr;
    cfg.numAttrs = best_ks > 1 ? 2 : 1;      // an unsplit launch keeps the plain block order (row blocks of a token tile run together)
    if (best_ks > 1) MDBF_CUDA(cudaLaunchKernelEx(&cfg, gemm_stage_kernel<LP, STAGE_A, true>, args, tm));
    else MDBF_CUDA(cudaLaunchKernelEx(&cfg, gemm_stage_kernel<LP, STAGE_A, false>, args, tm));
    return MDBF_OK;
}

template <int LP>
static mdbf_status_t run_prefill(Layer &L, const void *x, void *y, int T, cudaStream_t st) {
    const mdbf_desc_t &d = L.d;
    const int TT = PF_BN / LP;
    const int tok = T < TT ? T : TT;
    const int n_eff = ((tok * LP + 15) / 16) * 16;
    const int vec_ok = ((reinterpret_cast<uintptr_t>(x) & 15u) == 0 && d.d_in % 8 == 0) ? 1 : 0;
    {
        const bool few = (size_t)T * (L.padB / 8) < (size_t)148 * 256 * 4;     // few tokens: one thread per mode
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(pf_grid((size_t)T * (L.padB / 8) * (few ? LP : 1)));
        cfg.blockDim = dim3(256);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (few)
            MDBF_CUDA(cudaLaunchKernelEx(&cfg, prescale_kernel<LP, LP>, reinterpret_cast<const __nv_bfloat16 *>(x),
                                         (const float *)L.vtB, L.xsB, T, d.d_in, L.padB, vec_ok));
        else
            MDBF_CUDA(cudaLaunchKernelEx(&cfg, prescale_kernel<LP, 1>, reinterpret_cast<const __nv_bfloat16 *>(x),
                                         (const float *)L.vtB, L.xsB, T, d.d_in, L.padB, vec_ok));
    }
    MDBF_CUDA(cudaGetLastError());

    GemmArgs b = {};
    b.wk = L.wkB; b.rows_pad = L.rpB; b.rows = d.k; b.cols = d.d_in;
    b.U = L.UB; b.env_dtype = d.env_dtype; b.l = d.l; b.T = T; b.n_eff = n_eff;
    b.z = L.zsum; b.Vnext = L.VA; b.xs_next = L.xsA; b.pad_next = L.padA; b.status = L.status;
    const int bi = n_eff <= 64 ? 0 : n_eff <= 128 ? 1 : 2;    // narrowest TMA box that covers the used columns
    b.box_rows = 64 << bi;
    mdbf_status_t rc = launch_gemm<LP, false>(b, L.tmB[bi], st);
    if (rc) return rc;

    GemmArgs a = {};
    a.wk = L.wkA; a.rows_pad = L.rpA; a.rows = d.d_out; a.cols = d.k;
    a.U = L.UA; a.env_dtype = d.env_dtype; a.l = d.l; a.T = T; a.n_eff = n_eff;
    a.y = reinterpret_cast<__nv_bfloat16 *>(y); a.y32 = reinterpret_cast<float *>(y); a.y_mode = L.out_mode; a.status = L.status;
    a.box_rows = 64 << bi;
    return launch_gemm<LP, true>(a, L.tmA[bi], st);
}

// Scratch of the expanded order: the pre-scaled operands and their tensor maps.  Allocated on first use
// (mdbf_pack does it only for layers the materialised order cannot serve), which synchronises the device.
mdbf_status_t ensure_prefill_scratch(Layer &L) {
    if (L.xsB) return MDBF_OK;
    L.xs_rows = ((size_t)L.d.max_T * L.LP + 255) / 256 * 256;
    __nv_bfloat16 *b = nullptr, *a = nullptr;
    MDBF_CUDA(dev_malloc(&b, L.xs_rows * L.padB * 2));
    cudaError_t e = dev_malloc(&a, L.xs_rows * L.padA * 2);
    if (e == cudaSuccess) e = cudaMemset(b, 0, L.xs_rows * L.padB * 2);
    if (e == cudaSuccess) e = cudaMemset(a, 0, L.xs_rows * L.padA * 2);
    if (e != cudaSuccess) { cudaFree(b); cudaFree(a); return cuda_fail(e, "scratch of the expanded order"); }
    for (int i = 0; i < 3; ++i) {
        mdbf_status_t rc = make_xs_tensor_map(&L.tmB[i], b, L.xs_rows, L.padB, 64 << i);
        if (rc == MDBF_OK) rc = make_xs_tensor_map(&L.tmA[i], a, L.xs_rows, L.padA, 64 << i);
        if (rc) { cudaFree(b); cudaFree(a); return rc; }
    }
    L.xsB = b; L.xsA = a;
    return MDBF_OK;
}

mdbf_status_t launch_forward_prefill(Layer &L, const void *x, void *y, int T, cudaStream_t st, int *launches) {
    if (!L.xsB || !L.vtB || !L.wkB) {
        set_error("mdbf_linear_forward: the expanded-order kernel needs a layer packed with max_T >= 2");
        return MDBF_ERR_SHAPE;
    }
    mdbf_status_t rc;
    switch (L.LP) {
        case 1: rc = run_prefill<1>(L, x, y, T, st); break;
        case 2: rc = run_prefill<2>(L, x, y, T, st); break;
        case 4: rc = run_prefill<4>(L, x, y, T, st); break;
        case 8: rc = run_prefill<8>(L, x, y, T, st); break;
        case 16: rc = run_prefill<16>(L, x, y, T, st); break;
        case 32: rc = run_prefill<32>(L, x, y, T, st); break;
        default:
            set_error("mdbf_linear_forward: the large-T kernel handles l <= 32 (got %d)", L.d.l);
            return MDBF_ERR_SHAPE;
    }
    if (rc) return rc;
    L.last_ksplit = 0;
    *launches = 3;
    return MDBF_OK;
}

}  // namespace mdbf
