// Small-T path of the MDBF forward on the 5th-generation tensor cores, with the sign operand
// resident in tensor memory (TMEM).
//
// One stage is  out[tau][r] = sum_t U[r][t] * sum_c S[r][c] * V[c][t] * in[tau][c]
// (sum_t D_{u_t} S D_{v_t}, Eq. me-dbf-expand); stage B (S_B, V_B, U_B) maps x -> z, stage A
// (S_A, V_A, U_A) maps z -> y (Eq. DBF-inference-form, column convention).  As a contraction:
//
//     D[r][(tau, t)] = sum_c  A[r][c] * B[(tau, t)][c],   A = +-1.0 bf16 from the packed bits,
//                                                          B = bf16( V[c][t] * in[tau][c] )
//
// with N = LP * T <= 64 columns (LP = l rounded up to a power of two).  At such small N a
// tcgen05.mma lasts only N/2 .. 16 clocks, so two things decide the rate (measured): the A operand
// must not be re-read from shared memory for every instruction (4 KB per MMA), and one thread
// cannot issue MMAs faster than one per ~50 clocks.  Hence:
//
//   * A lives in TMEM.  Eight "expander" warps (thread = sign row = TMEM lane; warps w and w + 4
//     share a lane quadrant and take the even and the odd K blocks) read 64 packed bits per row and
//     K block, turn every bit into a +-1.0 bf16 with one shift and one logic op per two bits, and
//     write 32 TMEM columns with tcgen05.st; the store of one block overlaps the expansion of the
//     next.  Nothing of the expanded operand touches shared memory.
//   * Four issuer warps take the K blocks round-robin, each with its own fp32 accumulator in TMEM
//     (summed in the epilogue), so four MMAs are in flight at any time.  The same warps build
//     their B tiles (64 K x N, 128B-swizzled, K-major) in shared memory from the staged
//     activations and the 16-bit V block.
//   * Packed sign words (1 KB per K block) and V blocks stream in through cp.async.bulk into deep
//     mbarrier rings, requested before the programmatic-dependent-launch wait: they are immutable
//     weights, so with back-to-back launches they are in flight while the previous kernel drains.
//   * CTA = 128 sign rows x a slice of the reduction; the KS CTAs that share a row block form a
//     thread-block cluster and reduce their partial outputs through distributed shared memory,
//     so z and y are written once, deterministically, with no atomics and no extra launch.
//
// Column order inside a K block: register i of word w holds bits (i, i + 16) of that word, so MMA
// k index p of a 64-column block is canonical column 32*(p/32) + (p%32)/2 + 16*(p%2).  The private
// copy of V (vperm_kernel) and the B tile builder use the same order; the result does not depend
// on it.
//
// Every mbarrier wait is bounded; when one expires the kernel records MDBF_ERR_TIMEOUT, every role
// falls through to the common exit (cluster barriers included), TMEM is released and the kernel
// returns.  Every TMA and bulk copy targets the issuing CTA's own shared memory only.
#include <cooperative_groups.h>

#include "tmem_ptx.cuh"

namespace cg = cooperative_groups;

namespace mdbf {

constexpr int TM_EXPANDERS = 256;                      // two groups of 4 warps: even / odd K blocks
constexpr int TM_THREADS = TM_EXPANDERS + TM_ISSUERS * 32 + 64;   // + sign loader warp + V loader warp
constexpr int TM_W_ISSUER0 = TM_EXPANDERS / 32;        // first issuer warp
constexpr int TM_VSTAGES = 8;                          // V ring (two per issuer warp)
constexpr int TM_MAX_SSTAGES = 32;                     // sign ring, 1 KB per stage
constexpr int TM_MAX_ASTAGES = 12;                     // A stages in TMEM, 32 columns each (6 when TMEM is shared)
constexpr int TM_MAX_N = 64;
constexpr int TM_MAX_T = 16;

struct TmArgs {
    const uint2 *wk;          // K-blocked sign words [kblocks][rows_pad]
    int rows_pad;
    int rows, cols;
    const uint16_t *vperm;    // V in MMA k order, 16-bit env type: [kblocks][LP][64]
    const void *U;            // [rows][l] env_dtype
    int env_dtype, l;
    int T, n_mma;             // n_mma = T*LP rounded up to 16
    const void *in;           // stage B: bf16 x [T][cols]; stage A: fp32 z [T][cols]
    void *out;                // stage B: fp32 z [T][rows]; stage A: bf16 y [T][rows]
    int nkb_total;            // K blocks of 64 columns
    int kb_per_cta;           // K blocks per cluster rank
    int nastages;             // 4 or 8
    int nsstages;             // sign ring depth
    int tmem_cols;            // 256 or 512
    int32_t *status;
};


// Shared-memory plan (dynamic, 1024-byte aligned):
//   bbuf   [4 issuers][2][n_mma * 128 B]      B tiles
//   vring  [TM_VSTAGES][LP * 128 B]           V blocks (16-bit)
//   sring  [nsstages][1024 B]                 packed sign words of 128 rows x 64 columns
//   xin    [T][kb_per_cta * 64] float         staged activations of this CTA's reduction slice
//   part   [T][128] float                     this CTA's partial outputs (cluster reduction)
template <int LP, bool STAGE_A, bool ENV_BF16>
__global__ void __launch_bounds__(TM_THREADS, 1) tmem_stage_kernel(const TmArgs a) {
    using namespace tm;
    constexpr int MAXTOK = (TM_MAX_N / LP) < TM_MAX_T ? (TM_MAX_N / LP) : TM_MAX_T;
    extern __shared__ unsigned char tm_smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * TM_MAX_SSTAGES + 2 * TM_VSTAGES + 2 * TM_MAX_ASTAGES + 2 * TM_ISSUERS + 1];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;

    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(tm_smem_raw) + 1023u) & ~1023u;
    unsigned char *smem_gen = tm_smem_raw + (smem_base - smem_u32(tm_smem_raw));

    const int bbytes = a.n_mma * 128;
    const int vbytes = LP * 128;
    const int kslice = a.kb_per_cta * 64;
    const uint32_t off_v = (uint32_t)(TM_ISSUERS * 2 * bbytes);
    const uint32_t off_s = off_v + (uint32_t)(TM_VSTAGES * vbytes);
    const uint32_t off_x = off_s + (uint32_t)(a.nsstages * 1024);
    const uint32_t off_p = off_x + (uint32_t)(a.T * kslice * 4);
    float *xin = reinterpret_cast<float *>(smem_gen + off_x);
    float *part = reinterpret_cast<float *>(smem_gen + off_p);

    uint64_t *bp = bars;
    const uint32_t s_full = smem_u32(bp); bp += TM_MAX_SSTAGES;
    const uint32_t s_empty = smem_u32(bp); bp += TM_MAX_SSTAGES;
    const uint32_t v_full = smem_u32(bp); bp += TM_VSTAGES;
    const uint32_t v_empty = smem_u32(bp); bp += TM_VSTAGES;
    const uint32_t a_full = smem_u32(bp); bp += TM_MAX_ASTAGES;
    const uint32_t a_empty = smem_u32(bp); bp += TM_MAX_ASTAGES;
    const uint32_t b_empty = smem_u32(bp); bp += 2 * TM_ISSUERS;
    const uint32_t acc_bar = smem_u32(bp);

    const int row0 = blockIdx.x * 128;
    const int kb0 = blockIdx.y * a.kb_per_cta;
    const int nkb = max(0, min(a.kb_per_cta, a.nkb_total - kb0));
    const int nas = a.nastages, nss = a.nsstages;

    {   // one barrier per thread: s_full, s_empty, v_full, v_empty, a_full, a_empty, b_empty, acc_bar
        constexpr int NB0 = TM_MAX_SSTAGES, NB1 = 2 * TM_MAX_SSTAGES, NB2 = NB1 + TM_VSTAGES, NB3 = NB2 + TM_VSTAGES,
                      NB4 = NB3 + TM_MAX_ASTAGES, NB5 = NB4 + TM_MAX_ASTAGES, NB6 = NB5 + 2 * TM_ISSUERS;
        static_assert(NB6 + 1 <= TM_THREADS, "one thread per barrier");
        if (tid <= NB6) {
            const uint32_t count = tid < NB0 ? 1u : tid < NB1 ? 4u : tid < NB3 ? 1u : tid < NB4 ? 4u : tid < NB6 ? 1u
                                                                                                          : (uint32_t)TM_ISSUERS;
            mbar_init(smem_u32(&bars[tid]), count);
        }
        if (tid == 0) abort_flag_s = 0;
        fence_barrier_init();
    }
    if (warp == TM_W_ISSUER0) {
        tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)a.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    const uint32_t tmem_a0 = tmem + (uint32_t)(TM_ISSUERS * a.n_mma);     // first A stage column

    pdl_launch_dependents();

    float outv[MAXTOK];
#pragma unroll
    for (int i = 0; i < MAXTOK; ++i) outv[i] = 0.f;

    const int row_l = (warp & 3) * 32 + lane;               // row of the tile = TMEM lane (expander warps)
    if (warp < TM_W_ISSUER0) {
        // ============================ expanders, then epilogue ============================
        const int grp = warp >> 2;                           // 0: even K blocks (and the epilogue), 1: odd
        const int grow = row0 + row_l;
        float u[LP];
#pragma unroll
        for (int t = 0; t < LP; ++t)
            u[t] = (grp == 0 && grow < a.rows && t < a.l) ? env_load(a.U, (size_t)grow * a.l + t, a.env_dtype) : 0.f;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        bool alive = true;
        int rs = grp % nss, as = grp % nas;
        uint32_t rs_ph = 0, as_ph = 0;
        int prev_as = -1;
        for (int kb = grp; kb < nkb && alive; kb += 2) {
            alive = mbar_wait(s_full + 8 * rs, rs_ph, abort_flag, a.status);
            if (!alive) break;
            const uint2 w = *reinterpret_cast<const uint2 *>(smem_gen + off_s + rs * 1024 + row_l * 8);
            __syncwarp();
            if (lane == 0) mbar_arrive(s_empty + 8 * rs);
            uint32_t v[32];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                v[i] = ((w.x << (15 - i)) & 0x80008000u) | 0x3F803F80u;
                v[16 + i] = ((w.y << (15 - i)) & 0x80008000u) | 0x3F803F80u;
            }
            if (prev_as >= 0) {                              // the previous block's store had this long to land
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(a_full + 8 * prev_as);
            }
            alive = mbar_wait(a_empty + 8 * as, as_ph ^ 1u, abort_flag, a.status);
            if (!alive) break;
            tc_fence_after();
            tmem_st32(tmem_a0 + lane_base + (uint32_t)(as * 32), v);
            prev_as = as;
            rs += 2; if (rs >= nss) { rs -= nss; rs_ph ^= 1u; }
            as += 2; if (as >= nas) { as -= nas; as_ph ^= 1u; }
        }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (alive && prev_as >= 0 && lane == 0) mbar_arrive(a_full + 8 * prev_as);
        if (grp != 0) alive = false;                         // the odd group has no part in the epilogue
        if (alive) alive = mbar_wait(acc_bar, 0u, abort_flag, a.status);
        tc_fence_after();
        if (alive) {
            const int nacc = nkb < TM_ISSUERS ? nkb : TM_ISSUERS;
#pragma unroll
            for (int cc = 0; cc < TM_MAX_N / 16; ++cc) {
                if (cc * 16 < a.n_mma) {                                   // warp-uniform
                    float sum[16];
                    uint32_t d[TM_ISSUERS][16];
#pragma unroll
                    for (int acc = 0; acc < TM_ISSUERS; ++acc)
                        if (acc < nacc) tmem_ld16(tmem + lane_base + (uint32_t)(acc * a.n_mma + cc * 16), d[acc]);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        sum[j] = 0.f;
#pragma unroll
                        for (int acc = 0; acc < TM_ISSUERS; ++acc)
                            if (acc < nacc) sum[j] += __uint_as_float(d[acc][j]);
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int n = cc * 16 + j;
                        if (n / LP < MAXTOK) outv[n / LP] += u[n % LP] * sum[j];
                    }
                }
            }
        }
        if (grp == 0) {
#pragma unroll
            for (int tau = 0; tau < MAXTOK; ++tau)
                if (tau < a.T) part[tau * 128 + row_l] = outv[tau];
        }
    } else if (warp < TM_W_ISSUER0 + TM_ISSUERS) {
        // ===================== B-tile producers and MMA issuers ==========================
        const int w = warp - TM_W_ISSUER0;
        const int ptid = tid - TM_EXPANDERS;                 // 0..127 among the producer warps
        // B tiles start as zeros (rows beyond T*LP are never written again)
        for (int i = ptid; i < TM_ISSUERS * 2 * bbytes / 16; i += TM_ISSUERS * 32)
            reinterpret_cast<uint4 *>(smem_gen)[i] = make_uint4(0u, 0u, 0u, 0u);
        pdl_wait();                                          // the activations come from the previous kernel
        // stage in[tau][c0 .. c0 + kslice) as fp32, zero beyond the matrix; four columns per thread and step
        {
            const int c0 = kb0 * 64;
            const int quads = kslice >> 2;                   // kslice is a multiple of 64
            const int total = a.T * quads;
            const bool vec = (a.cols & 3) == 0 && (reinterpret_cast<uintptr_t>(a.in) & 15u) == 0;   // aligned rows
#pragma unroll 4
            for (int idx = ptid; idx < total; idx += TM_ISSUERS * 32) {
                const int tau = idx / quads, c = (idx - tau * quads) << 2;
                const int gc = c0 + c;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (vec && gc + 4 <= a.cols) {
                    if (STAGE_A) {
                        v = *reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(a.in) + (size_t)tau * a.cols + gc);
                    } else {
                        const uint2 r = *reinterpret_cast<const uint2 *>(reinterpret_cast<const __nv_bfloat16 *>(a.in) +
                                                                         (size_t)tau * a.cols + gc);
                        v = make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xFFFF0000u),
                                        __uint_as_float(r.y << 16), __uint_as_float(r.y & 0xFFFF0000u));
                    }
                } else {
                    float e[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        e[q] = 0.f;
                        if (gc + q < a.cols) {
                            if (STAGE_A) e[q] = reinterpret_cast<const float *>(a.in)[(size_t)tau * a.cols + gc + q];
                            else e[q] = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(a.in)[(size_t)tau * a.cols + gc + q]);
                        }
                    }
                    v = make_float4(e[0], e[1], e[2], e[3]);
                }
                *reinterpret_cast<float4 *>(xin + tau * kslice + c) = v;
            }
        }
        fence_proxy_async();                                 // the zeroed tiles are read by the tensor core
        asm volatile("bar.sync 1, 128;\n" ::: "memory");
        const uint32_t idesc = make_idesc(a.n_mma);
        const uint32_t d_tmem = tmem + (uint32_t)(w * a.n_mma);
        const int nchunks = a.T * LP * 8;                    // 16-byte chunks of real rows in a B tile
        bool alive = true;
        int it = 0;
        int as = w % nas;                                    // A stage of K block kb = w, w + 4, ...
        uint32_t as_ph = (uint32_t)(w / nas) & 1u;
        for (int kb = w; kb < nkb && alive; kb += TM_ISSUERS, ++it) {
            const int buf = it & 1, vs = kb % TM_VSTAGES;
            alive = mbar_wait(b_empty + 8 * (w * 2 + buf), ((uint32_t)(it >> 1) & 1u) ^ 1u, abort_flag, a.status);
            if (!alive) break;
            alive = mbar_wait(v_full + 8 * vs, (uint32_t)(kb / TM_VSTAGES) & 1u, abort_flag, a.status);
            if (!alive) break;
            unsigned char *bt = smem_gen + (size_t)(w * 2 + buf) * bbytes;
            const unsigned char *vb = smem_gen + off_v + vs * vbytes;
            const float *xk = xin + kb * 64;
#pragma unroll 4
            for (int i = lane; i < nchunks; i += 32) {
                const int n = i >> 3, j = i & 7;
                const int tau = n / LP, t = n % LP;
                const uint4 vv = *reinterpret_cast<const uint4 *>(vb + t * 128 + j * 16);
                const int b = 32 * (j >> 2) + 4 * (j & 3);
                const float4 xl = *reinterpret_cast<const float4 *>(xk + tau * kslice + b);
                const float4 xh = *reinterpret_cast<const float4 *>(xk + tau * kslice + b + 16);
                uint4 o;
                o.x = pack_bf16x2(env16<ENV_BF16>(vv.x & 0xFFFFu) * xl.x, env16<ENV_BF16>(vv.x >> 16) * xh.x);
                o.y = pack_bf16x2(env16<ENV_BF16>(vv.y & 0xFFFFu) * xl.y, env16<ENV_BF16>(vv.y >> 16) * xh.y);
                o.z = pack_bf16x2(env16<ENV_BF16>(vv.z & 0xFFFFu) * xl.z, env16<ENV_BF16>(vv.z >> 16) * xh.z);
                o.w = pack_bf16x2(env16<ENV_BF16>(vv.w & 0xFFFFu) * xl.w, env16<ENV_BF16>(vv.w >> 16) * xh.w);
                *reinterpret_cast<uint4 *>(bt + n * 128 + ((j ^ (n & 7)) << 4)) = o;
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(v_empty + 8 * vs);
            alive = mbar_wait(a_full + 8 * as, as_ph, abort_flag, a.status);
            if (!alive) break;
            tc_fence_after();
            if (lane == 0) {
                const uint64_t bdesc = make_smem_desc(smem_base + (uint32_t)((w * 2 + buf) * bbytes));
                const uint32_t a_t = tmem_a0 + (uint32_t)(as * 32);
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4)
                    umma_ts(d_tmem, a_t + (uint32_t)(8 * k4), bdesc + (uint64_t)(2 * k4), idesc, (it > 0 || k4 > 0) ? 1u : 0u);
                umma_commit(a_empty + 8 * as);
                umma_commit(b_empty + 8 * (w * 2 + buf));
            }
            __syncwarp();
            as += TM_ISSUERS;
            while (as >= nas) { as -= nas; as_ph ^= 1u; }
        }
        if (lane == 0) {
            if (alive && it > 0) umma_commit(acc_bar);       // arrives when this issuer's MMAs have retired
            else mbar_arrive(acc_bar);
        }
        __syncwarp();
    } else if (warp == TM_W_ISSUER0 + TM_ISSUERS) {
        // ============================== sign-word loader ================================
        if (lane == 0) {
            bool alive = true;
            for (int kb = 0; kb < nkb && alive; ++kb) {
                const int rs = kb % nss;
                alive = mbar_wait(s_empty + 8 * rs, ((uint32_t)(kb / nss) & 1u) ^ 1u, abort_flag, a.status);
                if (!alive) break;
                mbar_arrive_expect_tx(s_full + 8 * rs, 1024u);
                bulk_load(smem_base + off_s + (uint32_t)(rs * 1024), a.wk + (size_t)(kb0 + kb) * a.rows_pad + row0, 1024u,
                          s_full + 8 * rs);
            }
            if (!alive) drain_delay();
        }
        __syncwarp();
    } else {
        // ================================ V-block loader =================================
        if (lane == 0) {
            bool alive = true;
            for (int kb = 0; kb < nkb && alive; ++kb) {
                const int vs = kb % TM_VSTAGES;
                alive = mbar_wait(v_empty + 8 * vs, ((uint32_t)(kb / TM_VSTAGES) & 1u) ^ 1u, abort_flag, a.status);
                if (!alive) break;
                mbar_arrive_expect_tx(v_full + 8 * vs, (uint32_t)vbytes);
                bulk_load(smem_base + off_v + (uint32_t)(vs * vbytes), a.vperm + (size_t)(kb0 + kb) * LP * 64, (uint32_t)vbytes,
                          v_full + 8 * vs);
            }
            if (!alive) drain_delay();
        }
        __syncwarp();
    }

    // ------------------------------ cluster reduction and store ------------------------------
    tc_fence_before();
    cluster.sync();
    if (warp < 4 && cluster.block_rank() == 0) {
        const int tid_r = row_l;
        const unsigned nranks = cluster.num_blocks();
#pragma unroll
        for (int tau = 0; tau < MAXTOK; ++tau)
            if (tau < a.T) {
                float rv[8];
#pragma unroll
                for (unsigned rk = 1; rk < 8; ++rk)          // all remote loads in flight together
                    rv[rk] = rk < nranks ? cluster.map_shared_rank(part, rk)[tau * 128 + tid_r] : 0.f;
#pragma unroll
                for (unsigned rk = 1; rk < 8; ++rk) outv[tau] += rv[rk];
            }
        pdl_wait();                                          // order the stores after the previous kernel
        const int grow = row0 + tid_r;
        if (grow < a.rows && !*abort_flag) {
#pragma unroll
            for (int tau = 0; tau < MAXTOK; ++tau)
                if (tau < a.T) {
                    if (STAGE_A) reinterpret_cast<__nv_bfloat16 *>(a.out)[(size_t)tau * a.rows + grow] = __float2bfloat16_rn(outv[tau]);
                    else reinterpret_cast<float *>(a.out)[(size_t)tau * a.rows + grow] = outv[tau];
                }
        }
    }
    cluster.sync();
    if (warp == TM_W_ISSUER0) tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
}

// ----------------------------------------------------------- pack-time private copy
// V (cols x l, env_dtype, 16-bit) in MMA k order: out[(kb * LP + t) * 64 + p] = V[c][t] with
// c = kb*64 + 32*(p/32) + (p%32)/2 + 16*(p%2); zero for c >= cols or t >= l.
__global__ void vperm_kernel(const void *__restrict__ V, int cols, int l, int env_dtype, uint16_t *__restrict__ out,
                             int kblocks, int LP) {
    const size_t total = (size_t)kblocks * LP * 64;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int p = (int)(idx & 63);
        const int t = (int)((idx >> 6) % LP);
        const int kb = (int)((idx >> 6) / LP);
        const int c = kb * 64 + 32 * (p >> 5) + ((p & 31) >> 1) + 16 * (p & 1);
        uint16_t v = 0;
        if (c < cols && t < l) v = reinterpret_cast<const uint16_t *>(V)[(size_t)c * l + t];
        out[idx] = v;
    }
}

mdbf_status_t launch_vperm(const void *V, int cols, int l, int env_dtype, uint16_t *out, int kblocks, int LP,
                           cudaStream_t st) {
    const size_t total = (size_t)kblocks * LP * 64;
    int grid = (int)((total + 255) / 256);
    if (grid > 148 * 16) grid = 148 * 16;
    if (grid < 1) grid = 1;
    vperm_kernel<<<grid, 256, 0, st>>>(V, cols, l, env_dtype, out, kblocks, LP);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

// ---------------------------------------------------------------------- launch
struct TmPlan {
    int ks, kb_per_cta, nastages, nsstages, tmem_cols, n_mma;
    size_t smem;
};

// Cluster size along the reduction: fill the 148 SMs (one CTA each), keep the per-CTA prologue
// small against its share of K blocks, keep the staged activations inside shared memory.
static bool plan_stage(int rows, int cols, int LP, int T, TmPlan *p) {
    const int n_real = T * LP;
    if (n_real > TM_MAX_N || T > TM_MAX_T) return false;
    const int n_mma = ((n_real + 15) / 16) * 16;
    const int rb = ceil_div(rows, 128), nkb = ceil_div(cols, 64);
    // TMEM columns: one accumulator per issuer, then the A stages (32 columns each)
    const int acc_cols = TM_ISSUERS * n_mma;
    // Half of TMEM (256 columns) when at least four A stages fit beside the accumulators, so that two
    // CTAs - this kernel's and the next one's, started early - can share an SM; else all of it.
    const int tmem_cols = (acc_cols + 4 * 32 <= 256) ? 256 : 512;
    int nas = (tmem_cols - acc_cols) / 32;
    if (nas > TM_MAX_ASTAGES) nas = TM_MAX_ASTAGES;
    if (nas < 2) return false;
    long best_cost = -1;
    int best_ks = 0;
    for (int ks = 1; ks <= 8; ks *= 2) {
        const int per = ceil_div(nkb, ks);
        if (ks > 1 && per * (ks - 1) >= nkb) continue;                 // an empty rank: pointless split
        const size_t xbytes = (size_t)T * per * 64 * 4;
        if (xbytes > 64 * 1024) continue;
        const long waves = ceil_div(rb * ks, 148);
        const long cost = waves * (per + 16);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_ks = ks; }
    }
    if (best_ks == 0) return false;
    p->ks = best_ks;
    p->kb_per_cta = ceil_div(nkb, best_ks);
    p->nastages = nas;
    p->nsstages = p->kb_per_cta < TM_MAX_SSTAGES ? p->kb_per_cta : TM_MAX_SSTAGES;
    if (p->nsstages < 1) p->nsstages = 1;
    p->tmem_cols = tmem_cols;
    p->n_mma = n_mma;
    p->smem = 1024 + (size_t)TM_ISSUERS * 2 * n_mma * 128 + (size_t)TM_VSTAGES * LP * 128 + (size_t)p->nsstages * 1024 +
              (size_t)T * p->kb_per_cta * 64 * 4 + (size_t)T * 128 * 4;
    return p->smem <= 220 * 1024;
}

bool tmem_path_supports(const Layer &L, int T) {
    if (!L.wk2A || L.d.l > 32) return false;      // 16-bit envelopes, l <= 32 (the generic kernel's V copy is built on first use)
    TmPlan pb, pa;
    return plan_stage(L.d.k, L.d.d_in, L.LP, T, &pb) && plan_stage(L.d.d_out, L.d.k, L.LP, T, &pa);
}

template <int LP, bool STAGE_A, bool ENV_BF16>
static mdbf_status_t launch_tm(const TmArgs &a, const TmPlan &p, cudaStream_t st) {
    auto kern = tmem_stage_kernel<LP, STAGE_A, ENV_BF16>;
    static bool attr_set = false;
    if (!attr_set) {
        MDBF_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
        attr_set = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ceil_div(a.rows, 128), p.ks, 1);
    cfg.blockDim = dim3(TM_THREADS);
    cfg.dynamicSmemBytes = p.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = p.ks;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    MDBF_CUDA(cudaLaunchKernelEx(&cfg, kern, a));
    return MDBF_OK;
}

template <int LP, bool ENV_BF16>
static mdbf_status_t run_tm(Layer &L, const void *x, void *y, int T, cudaStream_t st) {
    const mdbf_desc_t &d = L.d;
    TmPlan pb, pa;
    if (!plan_stage(d.k, d.d_in, LP, T, &pb) || !plan_stage(d.d_out, d.k, LP, T, &pa)) {
        set_error("mdbf_linear_forward: the TMEM-operand kernel does not take l=%d, T=%d on this shape", d.l, T);
        return MDBF_ERR_SHAPE;
    }
    TmArgs b = {};
    b.wk = L.wkB; b.rows_pad = L.rpB; b.rows = d.k; b.cols = d.d_in;
    b.vperm = L.vpB; b.U = L.UB; b.env_dtype = d.env_dtype; b.l = d.l;
    b.T = T; b.n_mma = pb.n_mma; b.in = x; b.out = L.zsum;
    b.nkb_total = ceil_div(d.d_in, 64); b.kb_per_cta = pb.kb_per_cta;
    b.nastages = pb.nastages; b.nsstages = pb.nsstages; b.tmem_cols = pb.tmem_cols; b.status = L.status;
    mdbf_status_t rc = launch_tm<LP, false, ENV_BF16>(b, pb, st);
    if (rc) return rc;
    TmArgs s = {};
    s.wk = L.wkA; s.rows_pad = L.rpA; s.rows = d.d_out; s.cols = d.k;
    s.vperm = L.vpA; s.U = L.UA; s.env_dtype = d.env_dtype; s.l = d.l;
    s.T = T; s.n_mma = pa.n_mma; s.in = L.zsum; s.out = y;
    s.nkb_total = ceil_div(d.k, 64); s.kb_per_cta = pa.kb_per_cta;
    s.nastages = pa.nastages; s.nsstages = pa.nsstages; s.tmem_cols = pa.tmem_cols; s.status = L.status;
    return launch_tm<LP, true, ENV_BF16>(s, pa, st);
}

mdbf_status_t launch_forward_tmem(Layer &L, const void *x, void *y, int T, cudaStream_t st, int *launches) {
    if (!L.wk2A || (T > 1 && (!L.vpA || !L.wkA))) {
        set_error("mdbf_linear_forward: this layer holds no TMEM-operand copies (fp32 envelopes or l > 32)");
        return MDBF_ERR_SHAPE;
    }
    const bool bf = L.d.env_dtype == MDBF_BF16;
    mdbf_status_t rc;
    if (T == 1 && L.vxA && L.vxB) {
        rc = launch_forward_tmem_t1(L, x, y, st);
        if (rc) return rc;
        L.last_ksplit = 0;
        *launches = last_t1_launch_count();
        return MDBF_OK;
    }
#define MDBF_TM_CASE(lp) case lp: rc = bf ? run_tm<lp, true>(L, x, y, T, st) : run_tm<lp, false>(L, x, y, T, st); break;
    switch (L.LP) {
        MDBF_TM_CASE(1) MDBF_TM_CASE(2) MDBF_TM_CASE(4) MDBF_TM_CASE(8) MDBF_TM_CASE(16) MDBF_TM_CASE(32)
        default:
            set_error("mdbf_linear_forward: the TMEM-operand kernel handles l <= 32 (got %d)", L.d.l);
            return MDBF_ERR_SHAPE;
    }
#undef MDBF_TM_CASE
    if (rc) return rc;
    L.last_ksplit = 0;
    *launches = 2;
    return MDBF_OK;
}

// ------------------------------------------------------------------ self-test of the bounded wait
// One warp waits on an mbarrier that nothing ever arrives at, with the same bounded wait the
// forward kernels use: after the time limit it must record MDBF_ERR_TIMEOUT in the status word and
// return normally (no trap, the context stays usable).
__global__ void wait_timeout_selftest_kernel(int32_t *status) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag_s;
    if (threadIdx.x == 0) {
        tm::mbar_init(tm::smem_u32(&bar), 1);
        abort_flag_s = 0;
        tm::fence_barrier_init();
    }
    __syncthreads();
    tm::mbar_wait(tm::smem_u32(&bar), 0u, &abort_flag_s, status);
}

mdbf_status_t launch_wait_timeout_selftest(Layer &L, cudaStream_t st) {
    wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(L.status);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

}  // namespace mdbf
