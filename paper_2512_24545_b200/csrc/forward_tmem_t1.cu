// One-token (T = 1) path of the MDBF forward: tcgen05 MMA with the sign operand in tensor memory
// and the activation folded into it.
//
// One stage is  out[r] = sum_t U[r][t] * sum_c S[r][c] * V[c][t] * in[c]  (sum_t D_{u_t} S D_{v_t},
// Eq. me-dbf-expand); stage B (S_B, V_B, U_B) maps x -> z, stage A (S_A, V_A, U_A) maps z -> y
// (Eq. DBF-inference-form, column convention).  As a contraction
//
//     D[r][t] = sum_c  A[r][c] * B[t][c],    A[r][c] = bf16(in[c]) with the packed bit XOR-ed into its
//                                            sign (add/sub only: no multiply by the sign),
//                                            B[t][c] = bf16(V[c][t]).
//
// B is immutable, so the layer keeps it as ready-made 128B-swizzled K-major tile images
// (vtile_kernel) that a bulk copy drops straight into the B stage: no operand is built at run
// time except A, and everything but the activation slice is in flight before the
// programmatic-dependent-launch wait.
//
// What the measurements on this GPU say the kernel has to respect:
//   * tcgen05.mma with N = 16 lasts ~8 clocks but one thread issues at most one per ~50 clocks,
//     and with A in shared memory every MMA re-reads 4 KB: A lives in TMEM and four issuer warps
//     work round-robin, each on its own accumulator (summed in the epilogue).
//   * The bit -> bf16 step costs one shift and one logic op per two bits, and logic ops issue at
//     half rate: this, not HBM, bounds the big layers (<= 128 sign bits per clock and SM).
//   * A warp that walks one K block at a time spends most of its time in fixed latencies (every
//     mbarrier test ~100 clocks, every branch ~15): the unit of work is a PAIR of K blocks (128
//     columns, one 2 KB bulk copy of sign words, one 4 KB copy of V tiles, 64 TMEM columns, eight
//     MMAs, one commit), and TX_GROUPS groups of four expander warps work on different pairs at
//     the same time.
//
// CTA = 128 sign rows x a slice of the reduction; the KS CTAs of a row block form a cluster and
// reduce their partial outputs through distributed shared memory (deterministic, no atomics).
// Column order inside a K block: MMA k index p is canonical column
// 32*(p/32) + (p%32)/2 + 16*(p%2).  Every mbarrier wait is bounded (MDBF_ERR_TIMEOUT in the
// status word, all roles fall through, TMEM released).  Every bulk copy targets the issuing CTA's own shared memory only.
#include <cooperative_groups.h>
#include <cstdlib>

#include "tmem_ptx.cuh"

namespace cg = cooperative_groups;

namespace mdbf {

// expander groups of 4 warps (template parameter G of the kernel; group g takes the pairs g, g + G, ...): 2 for
// CTAs with few pairs (all latency, fewer warps start faster), 3 for long CTAs (+5 % on 70B-class layers; 4: worse)
constexpr int TX_ISSUERS = 4;                          // MMA issuer warps, one accumulator each (a thread issues ~1 MMA / 100+ clk here)
constexpr int tx_threads(int groups) { return groups * 128 + TX_ISSUERS * 32 + 64; }   // + sign loader warp + V loader warp
constexpr int TX_MAX_SSTAGES = 16;                     // sign ring: 2 KB per stage (one pair of K blocks)
constexpr int TX_MAX_ASTAGES = 7;                      // A / V stages: 64 TMEM columns + two V tiles each

struct TxArgs {
    const uint2 *wk2;         // sign words, row-block major: [row block][kb_pad][128 rows], 64 bits each
    int kb_pad;               // K blocks per row block in wk2 / vtile (even, zero padded)
    int rows, cols;
    int rb0;                  // first row block this launch serves in this layer (a launch may cover a slice of the row blocks)
    const uint16_t *vtile;    // bf16 V tile images [kb_pad][NB * 64], 128B-swizzled, NB = max(LP, 16)
    const void *U;            // [rows][l] env_dtype
    int env_dtype, l;
    const void *in;           // stage B: bf16 x [cols]; stage A: fp32 z [cols]
    void *out;                // stage B: fp32 z [rows]; stage A: bf16 y [rows]
    void *out_final;          // stage A, mode 4: bf16 y [rows] that receives round(out[] + this term)
    int npairs_total;         // pairs of K blocks along the reduction
    int pairs_per_cta;        // pairs per cluster rank
    int nastages, nsstages, tmem_cols;
    int stage_a;              // 0: stage B (bf16 in, fp32 out); stage A (fp32 in): 1 bf16 out, 2 fp32 out, 3 added to fp32 out,
                              // 4 last term of a sum: out_final = bf16(fp32 out + this term)
    int32_t *status;
};

// One launch may serve several layers that share their input (sibling projections: q/k/v, gate/up):
// the row blocks of the layers are laid side by side along blockIdx.x, the cluster size, ring depths
// and TMEM plan are common, everything else is per layer.
constexpr int TX_MAX_LAYERS = 4;
struct TxMulti {
    TxArgs layer[TX_MAX_LAYERS];
    int rb_start[TX_MAX_LAYERS + 1];   // first row block of each layer; rb_start[nlayers] = gridDim.x
    int nlayers;
};

// First test inline (the common case: the barrier has completed), bounded loop otherwise.
__device__ __forceinline__ bool tx_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *status) {
    if (tm::mbar_try_wait(bar, parity)) return true;
    return tm::mbar_wait(bar, parity, abort_flag, status);
}

// Shared-memory plan (dynamic, 1024-byte aligned):
//   vring [nastages][2 * NB * 128 B]   V tile images of a pair (B operand)
//   sring [nsstages][2048 B]           packed sign words of a pair: [2][128 rows] uint2
//   xp    [pairs_per_cta * 64] u32     activation pairs in MMA k order (bf16x2)
//   part  [8][128] float               partial outputs pushed by the other cluster ranks (rank 0 only reads)
template <int LP, int TX_GROUPS, bool SUM_LAST = false>
__device__ __forceinline__ void tmem_t1_body(const TxArgs &a, const int rb) {
    using namespace tm;
    constexpr int TX_EXPANDERS = TX_GROUPS * 128;
    constexpr int TX_W_ISSUER0 = TX_EXPANDERS / 32;
    constexpr int NB = LP < 16 ? 16 : LP;                    // MMA N
    constexpr int VBYTES = 2 * NB * 128;                     // two tiles
    extern __shared__ unsigned char tx_smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * TX_MAX_SSTAGES + 3 * TX_MAX_ASTAGES + 1];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;
    const bool stage_a = a.stage_a != 0;

    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(tx_smem_raw) + 1023u) & ~1023u;
    unsigned char *smem_gen = tx_smem_raw + (smem_base - smem_u32(tx_smem_raw));
    const int nas = a.nastages, nss = a.nsstages;
    const uint32_t off_s = (uint32_t)(nas * VBYTES);
    const uint32_t off_x = off_s + (uint32_t)(nss * 2048);
    const uint32_t off_p = off_x + (uint32_t)(a.pairs_per_cta * 256);
    uint32_t *xp = reinterpret_cast<uint32_t *>(smem_gen + off_x);
    float *part = reinterpret_cast<float *>(smem_gen + off_p);

    constexpr int NB0 = TX_MAX_SSTAGES, NB1 = 2 * TX_MAX_SSTAGES, NB2 = NB1 + TX_MAX_ASTAGES,
                  NB3 = NB2 + TX_MAX_ASTAGES, NB4 = NB3 + TX_MAX_ASTAGES;
    const uint32_t s_full = smem_u32(&bars[0]), s_empty = smem_u32(&bars[NB0]), v_full = smem_u32(&bars[NB1]),
                   a_full = smem_u32(&bars[NB2]), a_empty = smem_u32(&bars[NB3]), acc_bar = smem_u32(&bars[NB4]);

    const int row0 = rb * 128;
    const int pr0 = blockIdx.y * a.pairs_per_cta;
    const int npr = max(0, min(a.pairs_per_cta, a.npairs_total - pr0));

    if (tid <= NB4) {       // s_full 1, s_empty 4, v_full 1, a_full 4, a_empty 1, acc_bar TX_ISSUERS
        const uint32_t count = tid < NB0 ? 1u : tid < NB1 ? 4u : tid < NB2 ? 1u : tid < NB3 ? 4u : tid < NB4 ? 1u
                                                                                                      : (uint32_t)TX_ISSUERS;
        mbar_init(smem_u32(&bars[tid]), count);
    }
    if (tid == 0) abort_flag_s = 0;
    fence_barrier_init();
    if (warp == TX_W_ISSUER0) {
        tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)a.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    const uint32_t tmem_a0 = tmem + (uint32_t)(TX_ISSUERS * NB);

    pdl_launch_dependents();

    const int row_l = (warp & 3) * 32 + lane;                // row of the tile = TMEM lane (expander warps)
    float outv = 0.f;

    if (warp < TX_W_ISSUER0) {
        // ============================ expanders, then epilogue ============================
        const int grp = warp >> 2;
        const int grow = row0 + row_l;
        float u[LP];
#pragma unroll
        for (int t = 0; t < LP; ++t)
            u[t] = (grp == 0 && grow < a.rows && t < a.l) ? env_load(a.U, (size_t)grow * a.l + t, a.env_dtype) : 0.f;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;

        // stage the activation slice as bf16 pairs in MMA k order: pair `col` of a K block holds
        // columns 32*(col/16) + col%16 and that + 16; four pairs per thread and step
        pdl_wait();
        {
            const int c0 = pr0 * 128;
            const int quads = a.pairs_per_cta * 16;
            const bool vec = (a.cols & 3) == 0 && (reinterpret_cast<uintptr_t>(a.in) & 15u) == 0;
            for (int q = tid; q < quads; q += TX_EXPANDERS) {
                const int kbl = q >> 3, col = (q & 7) << 2;
                const int c_lo = c0 + kbl * 64 + 32 * (col >> 4) + (col & 15);
                float lo[4], hi[4];
                if (vec && c_lo + 20 <= a.cols) {
                    if (stage_a) {
                        const float4 l4 = *reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(a.in) + c_lo);
                        const float4 h4 = *reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(a.in) + c_lo + 16);
                        lo[0] = l4.x; lo[1] = l4.y; lo[2] = l4.z; lo[3] = l4.w;
                        hi[0] = h4.x; hi[1] = h4.y; hi[2] = h4.z; hi[3] = h4.w;
                    } else {
                        const uint2 l2 = *reinterpret_cast<const uint2 *>(reinterpret_cast<const __nv_bfloat16 *>(a.in) + c_lo);
                        const uint2 h2 = *reinterpret_cast<const uint2 *>(reinterpret_cast<const __nv_bfloat16 *>(a.in) + c_lo + 16);
                        lo[0] = __uint_as_float(l2.x << 16); lo[1] = __uint_as_float(l2.x & 0xFFFF0000u);
                        lo[2] = __uint_as_float(l2.y << 16); lo[3] = __uint_as_float(l2.y & 0xFFFF0000u);
                        hi[0] = __uint_as_float(h2.x << 16); hi[1] = __uint_as_float(h2.x & 0xFFFF0000u);
                        hi[2] = __uint_as_float(h2.y << 16); hi[3] = __uint_as_float(h2.y & 0xFFFF0000u);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int cl = c_lo + e, ch = c_lo + 16 + e;
                        lo[e] = 0.f; hi[e] = 0.f;
                        if (stage_a) {
                            if (cl < a.cols) lo[e] = reinterpret_cast<const float *>(a.in)[cl];
                            if (ch < a.cols) hi[e] = reinterpret_cast<const float *>(a.in)[ch];
                        } else {
                            if (cl < a.cols) lo[e] = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(a.in)[cl]);
                            if (ch < a.cols) hi[e] = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(a.in)[ch]);
                        }
                    }
                }
                *reinterpret_cast<uint4 *>(xp + kbl * 32 + col) =
                    make_uint4(pack_bf16x2(lo[0], hi[0]), pack_bf16x2(lo[1], hi[1]), pack_bf16x2(lo[2], hi[2]),
                               pack_bf16x2(lo[3], hi[3]));
            }
        }
        asm volatile("bar.sync 2, %0;\n" ::"n"(TX_EXPANDERS) : "memory");

        // One pair of K blocks per iteration: 2 x 64 sign bits of this row -> 64 TMEM columns.
        bool alive = true;
        int rs = grp % nss, as = grp % nas;
        uint32_t rs_ph = (uint32_t)(grp / nss) & 1u, as_ph = (uint32_t)(grp / nas) & 1u;
        int prev_as = -1;
        for (int pr = grp; pr < npr; pr += TX_GROUPS) {
            alive = tx_wait(s_full + 8 * rs, rs_ph, abort_flag, a.status);
            if (!alive) break;
            const unsigned char *sw = smem_gen + off_s + rs * 2048 + row_l * 8;
            const uint2 w0 = *reinterpret_cast<const uint2 *>(sw);
            const uint2 w1 = *reinterpret_cast<const uint2 *>(sw + 1024);
            __syncwarp();
            if (lane == 0) mbar_arrive(s_empty + 8 * rs);
            if (prev_as >= 0) {                              // retire the previous pair: its stores had an iteration to land
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(a_full + 8 * prev_as);
            }
            alive = tx_wait(a_empty + 8 * as, as_ph ^ 1u, abort_flag, a.status);
            if (!alive) break;
            tc_fence_after();
            const uint4 *xq = reinterpret_cast<const uint4 *>(xp + pr * 64);
            const uint32_t a_col = tmem_a0 + lane_base + (uint32_t)(as * 64);
#pragma unroll
            for (int q = 0; q < 8; ++q) {                    // TMEM columns 8q .. 8q+7 of the stage
                const uint32_t word = q < 2 ? w0.x : q < 4 ? w0.y : q < 6 ? w1.x : w1.y;
                const uint4 xa = xq[2 * q], xb = xq[2 * q + 1];
                const uint32_t xs8[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
                uint32_t v[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int i = (q & 1) * 8 + e;           // bits (i, i + 16) of the word
                    v[e] = ((word << (15 - i)) & 0x80008000u) ^ xs8[e];
                }
                tmem_st8(a_col + (uint32_t)(8 * q), v);
            }
            prev_as = as;
            rs += TX_GROUPS; while (rs >= nss) { rs -= nss; rs_ph ^= 1u; }
            as += TX_GROUPS; while (as >= nas) { as -= nas; as_ph ^= 1u; }
        }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (alive && prev_as >= 0 && lane == 0) mbar_arrive(a_full + 8 * prev_as);
        if (grp != 0) alive = false;                         // only the first group runs the epilogue
        if (alive) alive = mbar_wait(acc_bar, 0u, abort_flag, a.status);
        tc_fence_after();
        if (alive) {
            const int nacc = npr < TX_ISSUERS ? npr : TX_ISSUERS;
#pragma unroll
            for (int cc = 0; cc < NB / 16; ++cc) {
                float sum[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) sum[j] = 0.f;
#pragma unroll
                for (int a4 = 0; a4 < TX_ISSUERS; a4 += 4) {             // four accumulators per round of loads
                    uint32_t d[4][16];
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (a4 + q < nacc) tmem_ld16(tmem + lane_base + (uint32_t)((a4 + q) * NB + cc * 16), d[q]);
                    tmem_ld_wait();
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (a4 + q < nacc) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) sum[j] += __uint_as_float(d[q][j]);
                        }
                }
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (cc * 16 + j < LP) outv += u[(cc * 16 + j) % LP] * sum[j];
            }
        }
    }
    else if (warp < TX_W_ISSUER0 + TX_ISSUERS) {
        // ================================== MMA issuers ===================================
        const int w = warp - TX_W_ISSUER0;
        const uint32_t idesc = make_idesc(NB);
        const uint32_t d_tmem = tmem + (uint32_t)(w * NB);
        bool alive = true;
        int it = 0;
        int as = w % nas;
        uint32_t as_ph = (uint32_t)(w / nas) & 1u;
        // An issuer whose first pair already reuses a stage (w >= nas) has to see the earlier phases of
        // that stage complete first: a parity test alone cannot tell phase n from phase n - 2.
        if (w < npr)
            for (int k = 0; k < w / nas && alive; ++k) {
                alive = tx_wait(v_full + 8 * as, (uint32_t)k & 1u, abort_flag, a.status);
                if (alive) alive = tx_wait(a_full + 8 * as, (uint32_t)k & 1u, abort_flag, a.status);
            }
        for (int pr = w; pr < npr && alive; pr += TX_ISSUERS, ++it) {
            alive = tx_wait(v_full + 8 * as, as_ph, abort_flag, a.status);
            if (!alive) break;
            alive = tx_wait(a_full + 8 * as, as_ph, abort_flag, a.status);
            if (!alive) break;
            tc_fence_after();
            if (lane == 0) {
                const uint64_t bdesc = make_smem_desc(smem_base + (uint32_t)(as * VBYTES));
                const uint32_t a_t = tmem_a0 + (uint32_t)(as * 64);
#pragma unroll
                for (int k8 = 0; k8 < 8; ++k8)               // K block k8 / 4 of the pair, 16 k per MMA
                    umma_ts(d_tmem, a_t + (uint32_t)(8 * k8), bdesc + (uint64_t)((k8 >> 2) * (NB * 128 / 16) + 2 * (k8 & 3)), idesc,
                            (it > 0 || k8 > 0) ? 1u : 0u);
                umma_commit(a_empty + 8 * as);               // frees the A stage and the V stage together
            }
            __syncwarp();
            as += TX_ISSUERS;
            while (as >= nas) { as -= nas; as_ph ^= 1u; }
        }
        if (lane == 0) {
            if (alive && it > 0) umma_commit(acc_bar);       // arrives when this issuer's MMAs have retired
            else mbar_arrive(acc_bar);
        }
        __syncwarp();
    } else if (warp == TX_W_ISSUER0 + TX_ISSUERS) {
        // ============================== sign-word loader ================================
        if (lane == 0) {
            bool alive = true;
            int rs = 0;
            uint32_t ph = 0;
            const uint2 *src = a.wk2 + ((size_t)rb * a.kb_pad + (size_t)pr0 * 2) * 128;
            for (int pr = 0; pr < npr; ++pr) {
                alive = tx_wait(s_empty + 8 * rs, ph ^ 1u, abort_flag, a.status);
                if (!alive) break;
                mbar_arrive_expect_tx(s_full + 8 * rs, 2048u);
                bulk_load(smem_base + off_s + (uint32_t)(rs * 2048), src + (size_t)pr * 256, 2048u, s_full + 8 * rs);
                if (++rs == nss) { rs = 0; ph ^= 1u; }
            }
            if (!alive) drain_delay();
        }
        __syncwarp();
    } else {
        // ================================ V-tile loader ==================================
        if (lane == 0) {
            bool alive = true;
            int vs = 0;
            uint32_t ph = 0;
            const uint16_t *src = a.vtile + (size_t)pr0 * 2 * NB * 64;
            for (int pr = 0; pr < npr; ++pr) {
                alive = tx_wait(a_empty + 8 * vs, ph ^ 1u, abort_flag, a.status);
                if (!alive) break;
                mbar_arrive_expect_tx(v_full + 8 * vs, (uint32_t)VBYTES);
                bulk_load(smem_base + (uint32_t)(vs * VBYTES), src + (size_t)pr * 2 * NB * 64, (uint32_t)VBYTES, v_full + 8 * vs);
                if (++vs == nas) { vs = 0; ph ^= 1u; }
            }
            if (!alive) drain_delay();
        }
        __syncwarp();
    }

    // ------------------------------ cluster reduction and store ------------------------------
    // The other ranks push their partial outputs into rank 0's shared memory; one cluster barrier
    // (release / acquire) later rank 0 adds them up in rank order and stores.  Nobody reads a remote
    // CTA's memory after the barrier, so every CTA may leave as soon as it has passed it.
    tc_fence_before();
    const unsigned crank = cluster.block_rank();
    if (warp < 4 && crank != 0) cluster.map_shared_rank(part, 0)[crank * 128 + row_l] = outv;
    cluster.sync();
    if (warp < 4 && crank == 0) {
        const unsigned nranks = cluster.num_blocks();
#pragma unroll
        for (unsigned rk = 1; rk < 8; ++rk)
            if (rk < nranks) outv += part[rk * 128 + row_l];
        const int grow = row0 + row_l;
        if (grow < a.rows && !*abort_flag && store_in_bounds((size_t)grow, (size_t)a.rows, a.status)) {
            if (a.stage_a == 1) reinterpret_cast<__nv_bfloat16 *>(a.out)[grow] = __float2bfloat16_rn(outv);
            else if (a.stage_a == 3) reinterpret_cast<float *>(a.out)[grow] += outv;      // a further term of a sum of layers
            else if (SUM_LAST && a.stage_a == 4)                                           // its last term: one rounding of the whole sum
                reinterpret_cast<__nv_bfloat16 *>(a.out_final)[grow] = __float2bfloat16_rn(reinterpret_cast<const float *>(a.out)[grow] + outv);
            else reinterpret_cast<float *>(a.out)[grow] = outv;
        }
    }
    if (warp == TX_W_ISSUER0) tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
}

// One layer per launch: the arguments are plain kernel parameters (fastest for the small layers).
template <int LP, int G>
__global__ void __launch_bounds__(tx_threads(G), 1) tmem_t1_kernel(const TxArgs a) {
    tmem_t1_body<LP, G>(a, (int)blockIdx.x + a.rb0);
}

// The last term of a sum of layers (mode 4 of the epilogue), an instantiation of its own so that the plain kernel
// carries no trace of it.
template <int LP, int G>
__global__ void __launch_bounds__(tx_threads(G), 1) tmem_t1_sumlast_kernel(const TxArgs a) {
    tmem_t1_body<LP, G, true>(a, (int)blockIdx.x + a.rb0);
}

// Several sibling layers per launch: each CTA picks its layer by its position in the grid.
template <int LP, int G>
__global__ void __launch_bounds__(tx_threads(G), 1) tmem_t1_multi_kernel(const __grid_constant__ TxMulti m) {
    int li = 0;
#pragma unroll
    for (int i = 1; i < TX_MAX_LAYERS; ++i)
        if (i < m.nlayers && (int)blockIdx.x >= m.rb_start[i]) li = i;
    const TxArgs a = m.layer[li];                             // by value: one indexed read of the parameter block
    tmem_t1_body<LP, G>(a, (int)blockIdx.x - m.rb_start[li] + a.rb0);
}

// ----------------------------------------------------------- pack-time private copies
// bf16 V tile images: K block kb is NB rows (modes) x 64 k, K-major with 128-byte rows and the 128B
// swizzle; element (t, p) holds V[c][t], c = kb*64 + 32*(p/32) + (p%32)/2 + 16*(p%2), at 16-bit
// index kb*NB*64 + t*64 + ((p/8) ^ (t%8))*8 + p%8; zero outside the matrix (kblocks may exceed it).
__global__ void vtile_kernel(const void *__restrict__ V, int cols, int l, int env_dtype, uint16_t *__restrict__ out,
                             int kblocks, int NB) {
    const size_t total = (size_t)kblocks * NB * 64;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int p = (int)(idx & 63);
        const int t = (int)((idx >> 6) % NB);
        const int kb = (int)((idx >> 6) / NB);
        const int c = kb * 64 + 32 * (p >> 5) + ((p & 31) >> 1) + 16 * (p & 1);
        float v = 0.f;
        if (c < cols && t < l) v = env_load(V, (size_t)c * l + t, env_dtype);
        const __nv_bfloat16 b = __float2bfloat16_rn(v);
        out[(size_t)kb * NB * 64 + t * 64 + (((p >> 3) ^ (t & 7)) << 3) + (p & 7)] = *reinterpret_cast<const uint16_t *>(&b);
    }
}

// Row-block-major sign words: out[(rb * kb_pad + kb) * 128 + r] = canonical words (2kb, 2kb+1) of row
// rb*128 + r, zero (= +1) outside the matrix, so that a CTA's slice of the reduction is contiguous.
__global__ void wk2_kernel(const uint32_t *__restrict__ canon, int rows, int nwords, uint2 *__restrict__ out, int rblocks,
                           int kb_pad) {
    const size_t total = (size_t)rblocks * kb_pad * 128;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (size_t)gridDim.x * blockDim.x) {
        const int r = (int)(idx & 127);
        const int kb = (int)((idx >> 7) % kb_pad);
        const int rb = (int)((idx >> 7) / kb_pad);
        const int row = rb * 128 + r;
        uint2 v = make_uint2(0u, 0u);
        if (row < rows) {
            if (2 * kb < nwords) v.x = canon[(size_t)row * nwords + 2 * kb];
            if (2 * kb + 1 < nwords) v.y = canon[(size_t)row * nwords + 2 * kb + 1];
        }
        out[idx] = v;
    }
}

static int tx_grid(size_t items) {
    size_t g = (items + 255) / 256;
    if (g < 1) g = 1;
    if (g > 148 * 16) g = 148 * 16;
    return (int)g;
}

mdbf_status_t launch_vtile(const void *V, int cols, int l, int env_dtype, uint16_t *out, int kblocks, int NB,
                           cudaStream_t st) {
    vtile_kernel<<<tx_grid((size_t)kblocks * NB * 64), 256, 0, st>>>(V, cols, l, env_dtype, out, kblocks, NB);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

mdbf_status_t launch_wk2(const uint32_t *canon, int rows, int nwords, uint2 *out, int rblocks, int kb_pad,
                         cudaStream_t st) {
    wk2_kernel<<<tx_grid((size_t)rblocks * kb_pad * 128), 256, 0, st>>>(canon, rows, nwords, out, rblocks, kb_pad);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

// ---------------------------------------------------------------------- launch
struct TxPlan {
    int ks, nastages, tmem_cols;
    int pairs_per_cta[TX_MAX_LAYERS], nsstages;
    size_t smem;
};

// Fixed part of a CTA's time (set-up, cluster reduction) in units of one K block of streaming (swept on the
// 7B- and 70B-class shapes).
static int fixed_cost() { return 48; }

// One plan for all the layers of a launch.  Cluster size along the reduction: one CTA per SM (all of
// TMEM), as few waves as possible, the per-CTA fixed part weighed against its share of the reduction.
static bool plan_t1(int n, const int *rows, const int *kb_pad, int LP, TxPlan *p) {
    const int NB = LP < 16 ? 16 : LP;
    int nas = (512 - TX_ISSUERS * NB) / 64;
    if (nas > TX_MAX_ASTAGES) nas = TX_MAX_ASTAGES;
    const int max_ks = 8;                                     // portable cluster size
    int rb = 0, max_pairs = 0, min_pairs = 1 << 30;
    for (int i = 0; i < n; ++i) {
        rb += ceil_div(rows[i], 128);
        max_pairs = max(max_pairs, kb_pad[i] / 2);
        min_pairs = min(min_pairs, kb_pad[i] / 2);
    }
    long best_cost = -1;
    int best_ks = 1;
    for (int ks = 1; ks <= max_ks; ks *= 2) {
        if (ks > 1 && ceil_div(min_pairs, ks) * (ks - 1) >= min_pairs) continue;     // an empty rank in some layer
        const long waves = ceil_div(rb * ks, 148);
        const long cost = waves * (2 * ceil_div(max_pairs, ks) + fixed_cost());
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_ks = ks; }
    }
    p->ks = best_ks;
    int max_per = 1;
    for (int i = 0; i < n; ++i) {
        p->pairs_per_cta[i] = ceil_div(kb_pad[i] / 2, best_ks);
        max_per = max(max_per, p->pairs_per_cta[i]);
    }
    p->nastages = nas;
    p->nsstages = max_per < TX_MAX_SSTAGES ? max_per : TX_MAX_SSTAGES;
    p->tmem_cols = 512;
    p->smem = 1024 + (size_t)nas * 2 * NB * 128 + (size_t)p->nsstages * 2048 + (size_t)max_per * 256 + 4096;
    return nas >= 2 && p->smem <= 220 * 1024;
}

static thread_local int g_t1_launches = 0;      // kernels the last one-token forward of this thread launched
int last_t1_launch_count() { return g_t1_launches; }

template <int LP, int G>
static mdbf_status_t launch_t1g(const TxMulti &m, const TxPlan &p, cudaStream_t st) {
    static PerDeviceOnce once;
    if (once.first()) {
        MDBF_CUDA(cudaFuncSetAttribute(tmem_t1_kernel<LP, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
        MDBF_CUDA(cudaFuncSetAttribute(tmem_t1_multi_kernel<LP, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
        MDBF_CUDA(cudaFuncSetAttribute(tmem_t1_sumlast_kernel<LP, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(m.rb_start[m.nlayers], p.ks, 1);
    cfg.blockDim = dim3(tx_threads(G));
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
    if (m.nlayers == 1 && m.layer[0].stage_a == 4) MDBF_CUDA(cudaLaunchKernelEx(&cfg, tmem_t1_sumlast_kernel<LP, G>, m.layer[0]));
    else if (m.nlayers == 1) MDBF_CUDA(cudaLaunchKernelEx(&cfg, tmem_t1_kernel<LP, G>, m.layer[0]));
    else MDBF_CUDA(cudaLaunchKernelEx(&cfg, tmem_t1_multi_kernel<LP, G>, m));
    ++g_t1_launches;
    return MDBF_OK;
}
// Two expander groups for CTAs with few pairs of K blocks, three from `long_cta` pairs per CTA on (16: the
// 4096 x 4096 layers keep two groups, the 11008- and 70B-class layers get three).
template <int LP>
static mdbf_status_t launch_t1(const TxMulti &m, const TxPlan &p, cudaStream_t st) {
    const int long_cta = 16;
    int max_per = 0;
    for (int i = 0; i < m.nlayers; ++i) max_per = max(max_per, p.pairs_per_cta[i]);
    return max_per >= long_cta ? launch_t1g<LP, 3>(m, p, st) : launch_t1g<LP, 2>(m, p, st);
}

// One stage.  When the grid ends in a wave with only a few CTAs (448 row blocks on 148 SMs: the last 4 would
// cost a whole wave), those row blocks go to a second, short launch that splits their reduction over a
// cluster instead; both launches read the same input and write disjoint rows.
template <int LP>
static mdbf_status_t launch_stage(const TxMulti &full, const TxPlan &p, const int *kb_pad, cudaStream_t st) {
    const int n = full.nlayers, R = full.rb_start[n];
    int max_per = 0;
    for (int i = 0; i < n; ++i) max_per = max(max_per, p.pairs_per_cta[i]);
    const int tail = R % 148;                                   // CTAs of the last wave (cluster size 1)
    if (!(p.ks == 1 && R > 148 && tail > 0 && 4 * tail <= 148 && max_per >= 16)) return launch_t1<LP>(full, p, st);

    TxMulti part[2] = {};
    int rows_tail[TX_MAX_LAYERS], kb_tail[TX_MAX_LAYERS], src_tail[TX_MAX_LAYERS];
    const int cut = R - tail;                                   // global row blocks [0, cut) stay in the main launch
    for (int i = 0; i < n; ++i) {
        const int lo = full.rb_start[i], hi = full.rb_start[i + 1];
        for (int h = 0; h < 2; ++h) {
            const int a = max(lo, h ? cut : 0), b = min(hi, h ? R : cut);
            if (a >= b) continue;
            TxMulti &m = part[h];
            TxArgs &t = m.layer[m.nlayers];
            t = full.layer[i];
            t.rb0 = a - lo;
            if (h) { rows_tail[m.nlayers] = (b - a) * 128; kb_tail[m.nlayers] = kb_pad[i]; src_tail[m.nlayers] = i; }
            m.rb_start[m.nlayers + 1] = m.rb_start[m.nlayers] + (b - a);
            ++m.nlayers;
        }
    }
    TxPlan pt;
    if (!plan_t1(part[1].nlayers, rows_tail, kb_tail, LP, &pt)) return launch_t1<LP>(full, p, st);
    for (int j = 0; j < part[1].nlayers; ++j) {
        TxArgs &t = part[1].layer[j];
        t.pairs_per_cta = pt.pairs_per_cta[j];
        t.nastages = pt.nastages; t.nsstages = pt.nsstages; t.tmem_cols = pt.tmem_cols;
        (void)src_tail[j];
    }
    mdbf_status_t rc = launch_t1<LP>(part[0], p, st);
    if (rc) return rc;
    return launch_t1<LP>(part[1], pt, st);
}

// Both stages of n layers that read the same x (n = 1: a single layer): one launch per stage.
// sum != nullptr: the n layers are the terms of a sum; stage B of all terms shares one launch (they read the
// same x), the stage-A launches follow one another: term 0 stores its fp32 output into sum_acc, the middle
// terms add to it, the last one adds and rounds into sum_y.
template <int LP>
static mdbf_status_t run_t1(Layer *const *Ls, int n, const void *x, void *const *ys, cudaStream_t st,
                            float *sum_acc = nullptr, void *sum_y = nullptr, int stages = 3) {
    int rowsB[TX_MAX_LAYERS], kbB[TX_MAX_LAYERS], rowsA[TX_MAX_LAYERS], kbA[TX_MAX_LAYERS];
    for (int i = 0; i < n; ++i) {
        rowsB[i] = Ls[i]->d.k; kbB[i] = Ls[i]->kbpB;
        rowsA[i] = Ls[i]->d.d_out; kbA[i] = Ls[i]->kbpA;
    }
    g_t1_launches = 0;
    TxPlan pb, pa;
    if (!plan_t1(n, rowsB, kbB, LP, &pb) || !plan_t1(n, rowsA, kbA, LP, &pa)) {
        set_error("mdbf_linear_forward: the one-token TMEM kernel does not fit this shape");
        return MDBF_ERR_SHAPE;
    }
    TxMulti mb = {}, ma = {};
    mb.nlayers = ma.nlayers = n;
    for (int i = 0; i < n; ++i) {
        Layer &L = *Ls[i];
        const mdbf_desc_t &d = L.d;
        TxArgs &b = mb.layer[i];
        b.wk2 = L.wk2B; b.kb_pad = L.kbpB; b.rows = d.k; b.cols = d.d_in;
        b.vtile = L.vxB; b.U = L.UB; b.env_dtype = d.env_dtype; b.l = d.l;
        b.in = x; b.out = L.zsum; b.stage_a = 0;
        b.npairs_total = L.kbpB / 2; b.pairs_per_cta = pb.pairs_per_cta[i];
        b.nastages = pb.nastages; b.nsstages = pb.nsstages; b.tmem_cols = pb.tmem_cols; b.status = L.status;
        mb.rb_start[i + 1] = mb.rb_start[i] + ceil_div(d.k, 128);
        TxArgs &s = ma.layer[i];
        s.wk2 = L.wk2A; s.kb_pad = L.kbpA; s.rows = d.d_out; s.cols = d.k;
        s.vtile = L.vxA; s.U = L.UA; s.env_dtype = d.env_dtype; s.l = d.l;
        s.in = L.zsum; s.out = ys[i]; s.out_final = nullptr; s.stage_a = 1 + L.out_mode;
        s.npairs_total = L.kbpA / 2; s.pairs_per_cta = pa.pairs_per_cta[i];
        s.nastages = pa.nastages; s.nsstages = pa.nsstages; s.tmem_cols = pa.tmem_cols; s.status = L.status;
        ma.rb_start[i + 1] = ma.rb_start[i] + ceil_div(d.d_out, 128);
    }
    mdbf_status_t rc = (stages & 1) ? launch_stage<LP>(mb, pb, kbB, st) : MDBF_OK;     // stages: bit 0 = stage B, bit 1 = stage A
    if (rc) return rc;
    if (!(stages & 2)) return MDBF_OK;
    if (!sum_acc) return launch_stage<LP>(ma, pa, kbA, st);
    for (int i = 0; i < n; ++i) {
        TxMulti one = {};
        one.nlayers = 1;
        one.rb_start[1] = ceil_div(rowsA[i], 128);
        TxPlan p1;
        if (!plan_t1(1, &rowsA[i], &kbA[i], LP, &p1)) {
            set_error("mdbf_linear_forward_sum: the one-token TMEM kernel does not fit this shape");
            return MDBF_ERR_SHAPE;
        }
        TxArgs &s = one.layer[0];
        s = ma.layer[i];
        s.out = n == 1 ? sum_y : (void *)sum_acc;
        s.out_final = sum_y;
        s.stage_a = n == 1 ? 1 : i == 0 ? 2 : i == n - 1 ? 4 : 3;
        s.pairs_per_cta = p1.pairs_per_cta[0];
        s.nastages = p1.nastages; s.nsstages = p1.nsstages; s.tmem_cols = p1.tmem_cols;
        rc = launch_stage<LP>(one, p1, &kbA[i], st);
        if (rc) return rc;
    }
    return MDBF_OK;
}

// n <= TX_MAX_LAYERS layers with the same LP, all prepared for the one-token kernel.
mdbf_status_t launch_forward_tmem_t1_multi(Layer *const *Ls, int n, const void *x, void *const *ys, cudaStream_t st, int stages) {
    switch (Ls[0]->LP) {
        case 1: return run_t1<1>(Ls, n, x, ys, st, nullptr, nullptr, stages);
        case 2: return run_t1<2>(Ls, n, x, ys, st, nullptr, nullptr, stages);
        case 4: return run_t1<4>(Ls, n, x, ys, st, nullptr, nullptr, stages);
        case 8: return run_t1<8>(Ls, n, x, ys, st, nullptr, nullptr, stages);
        case 16: return run_t1<16>(Ls, n, x, ys, st, nullptr, nullptr, stages);
        case 32: return run_t1<32>(Ls, n, x, ys, st, nullptr, nullptr, stages);
        default:
            set_error("mdbf_linear_forward: the one-token TMEM kernel handles l <= 32 (got %d)", Ls[0]->d.l);
            return MDBF_ERR_SHAPE;
    }
}

// The terms of a sum of layers (same LP, at most TX_MAX_LAYERS) at one token: y = bf16(sum of the terms' outputs).
mdbf_status_t launch_forward_tmem_t1_sum(Layer *const *Ls, int n, const void *x, float *acc, void *y, cudaStream_t st) {
    void *ys[TX_MAX_LAYERS] = {};
    switch (Ls[0]->LP) {
        case 1: return run_t1<1>(Ls, n, x, ys, st, acc, y);
        case 2: return run_t1<2>(Ls, n, x, ys, st, acc, y);
        case 4: return run_t1<4>(Ls, n, x, ys, st, acc, y);
        case 8: return run_t1<8>(Ls, n, x, ys, st, acc, y);
        case 16: return run_t1<16>(Ls, n, x, ys, st, acc, y);
        case 32: return run_t1<32>(Ls, n, x, ys, st, acc, y);
        default:
            set_error("mdbf_linear_forward_sum: the one-token TMEM kernel handles l <= 32 (got %d)", Ls[0]->d.l);
            return MDBF_ERR_SHAPE;
    }
}

// Whether the one-token TMEM-operand kernel can run this layer (16-bit envelopes, l <= 32, both stages plannable).
bool tmem_path_supports(const Layer &L, int T) {
    if (T != 1 || !L.wk2A || !L.vxA || !L.vxB || L.d.l > 32) return false;
    const int rowsB = L.d.k, rowsA = L.d.d_out;
    TxPlan pb, pa;
    return plan_t1(1, &rowsB, &L.kbpB, L.LP, &pb) && plan_t1(1, &rowsA, &L.kbpA, L.LP, &pa);
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

mdbf_status_t launch_forward_tmem(Layer &L, const void *x, void *y, int T, cudaStream_t st, int *launches) {
    if (T != 1 || !L.wk2A || !L.vxA || !L.vxB) {
        set_error("mdbf_linear_forward: the TMEM-operand kernel takes one token, 16-bit envelopes and l <= 32");
        return MDBF_ERR_SHAPE;
    }
    mdbf_status_t rc = launch_forward_tmem_t1(L, x, y, st);
    if (rc) return rc;
    L.last_ksplit = 0;
    *launches = last_t1_launch_count();
    return MDBF_OK;
}

mdbf_status_t launch_forward_tmem_t1(Layer &L, const void *x, void *y, cudaStream_t st) {
    Layer *one[1] = {&L};
    void *ys[1] = {y};
    return launch_forward_tmem_t1_multi(one, 1, x, ys, st, 3);
}

}  // namespace mdbf
