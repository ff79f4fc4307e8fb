// One-token (T = 1) path of the MDBF forward: integer tensor-core contraction with the packed sign bits,
// one byte each, as the A operand; four short launches per forward, none of which waits on another CTA.
//
// One stage is  out[r] = sum_t U[r][t] * sum_c S[r][c] * V[c][t] * in[c]   (sum_t D_{u_t} S D_{v_t},
// Eq. me-dbf-expand); stage B (S_B, V_B, U_B) maps x -> z, stage A (S_A, V_A, U_A) maps z -> y
// (Eq. DBF-inference-form, column convention).
//
// The scaled operand w[c][t] = V[c][t] * in[c] (the first step of a stage: the pre-scale by the envelope
// factor) is turned into a 21-bit fixed-point number per mode t,  w ~ delta_t * q,  |q| <= 2^20 - 2,
// q = q0 + 2^7 q1 + 2^14 q2  with three signed 8-bit digits, delta_t from max|in| * max_c |V[c][t]|.
// The contraction with the signs is then an exact integer matrix product
//
//     D[r][(j, t)] = sum_c 128 b[r][c] * q_j[c][t]      tcgen05.mma kind::i8, M = 128, N = 3 * l, K = 32
//
// whose A operand costs one left shift (a multiply: FMA pipe) and one AND (ALU pipe) per FOUR sign bits:
// (word << (7 - i)) & 0x80808080 is four unsigned bytes 128 b (b = the packed bit, set <=> sign -1),
// stored to tensor memory as they are, and with S = 1 - 2 b
//
//     sum_c S[r][c] q[c][t] = sum_c q[c][t]  -  2 * sum_c b[r][c] q[c][t]
//
// the row-independent first term (column sums of q, stored per pair of K blocks beside the images) is added by
// every segment for the pairs it covers.  The accumulators are int32 and exact, so the only roundings
// of the path are the fixed-point step (2^-21 of the operand's range) and the final store.  The B operand
// ("image" of a pair of K blocks: N rows x 128 bytes, K-major, 128B swizzle) is built once per stage and
// shared by every row block.
//
// Launch structure, per forward of one or several layers (programmatic dependent launches):
//
//     image kernel (x)  ->  stage kernel B: z, max|z|  ->  image kernel (z)  ->  stage kernel A: y
//
// image kernel: one CTA per pair of K blocks of every layer: max |input|, fixed-point digits, column sums.
// stage kernel: a fixed grid of CTAs (one per SM), each walking its share of the units (group of four row
// blocks of 128 rows) x (pair of K blocks) of every layer, in layer order.  Roles of a CTA: four groups of
// four expander warps (group = row block of the unit, thread = row = TMEM lane), eight MMA issuer warps (two
// per row block, one for the even and one for the odd units, i.e. one per A stage of the row block; both add
// into the row block's accumulator), one warp bulk-copying sign words (ring of 8 units = 64 KB, lane = ring
// slot), one bulk-copying images (ring of 8), and four epilogue
// warps (tcgen05.ld, contraction with U).  A group of row blocks split over several CTAs is summed through
// one 64-bit integer atomic per row (order-independent, hence deterministic): the thread whose addition
// completes the row's count finalises the row.  No CTA ever waits for another one; every mbarrier wait is
// bounded, and on expiry the status words read MDBF_ERR_TIMEOUT, all roles fall through and TMEM is
// released.  Every bulk copy targets the issuing CTA's own shared memory.
#include <cstdlib>

#include "tmem_ptx.cuh"

namespace mdbf {
namespace t1 {

constexpr int kMaxLayers = 8;
constexpr float kQmax = 1048574.f;                 // 2^20 - 2: range of the fixed-point operand
constexpr int kRBG = 4;                            // row blocks per unit (they share the unit's image)
constexpr int kSignSlots = 8;                      // sign ring: 8 KB per slot (four row blocks x one pair of K blocks)
constexpr int kImgSlots = 8;                       // image ring
constexpr int kIssuers = 8;                        // two per row block of the unit: even and odd units
constexpr int kThreads = (4 * 4 + 4 + kIssuers + 2) * 32;
constexpr int kImgThreads = 512;                   // image kernel: 128 builders, all of them for the pass over the input

// word offsets inside a layer's scalar block (uint32 words)
constexpr int kSyAmax = 0;                         // [2] float bits: max |input| of the stage (stage B: max |x|, stage A: max |z|)
constexpr int kSyWords = 2;

struct Stage {
    const uint2 *wk2;          // sign words [R][kb_pad][128 rows], 64 bits each
    const void *V;             // [cols][l] 16-bit envelope factor the input is scaled by
    const void *U;             // [rows][l] 16-bit envelope factor the modes are contracted with
    const float *vmax;         // [32] max_c |V[c][t]|
    int8_t *img;               // [Np][NB][128] operand images (scratch, rewritten by every launch)
    int *colsum;               // [Np][32] column sums of q per pair and mode (scratch, rewritten with the images)
    unsigned long long *acc64; // [R * 128] fixed-point sums of the partial outputs of split groups (zero between launches)
    int rows, cols;
    int R, RG, Np, kb_pad;
    int unit0;                 // first unit of this stage of this layer among the launch's units of the stage
    int item0;                 // first image of this stage of this layer among the launch's images of the stage
};

struct LayerArgs {
    Stage st[2];               // 0: stage B (x -> z), 1: stage A (z -> y)
    const void *x;             // bf16 [d_in]
    float *z;                  // fp32 [k]
    void *y;                   // [d_out]
    unsigned int *sync;
    int32_t *status;
    int l, env_dtype, out_mode;    // out_mode 0: y bf16; 1: y fp32 stored; 2: y fp32 added to
};

struct Group {
    LayerArgs layer[kMaxLayers];
    int nlayers;
    int items[2];              // images per stage, all layers
    int units[2], chunk[2];    // units per stage, all layers; units per CTA
    unsigned shl_mul[8];       // 2^(7 - i): the expanders' left shifts as multiplies by a kernel parameter (FMA pipe, not the ALU pipe)
};

// ------------------------------------------------------------------ small device helpers
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;\n" ::: "memory"); }

__device__ __forceinline__ bool bwait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *status) {
    if (tm::mbar_try_wait(bar, parity)) return true;
    return tm::mbar_wait(bar, parity, abort_flag, status);
}

// D[tmem] (+)= A[tmem] * B[smem], 8-bit integer operands, int32 accumulator
__device__ __forceinline__ void umma_ts_i8(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// instruction descriptor: int32 accumulator, A unsigned and B signed 8-bit, both K-major, M = 128
__device__ __forceinline__ uint32_t make_idesc_i8(int n) {
    uint32_t d = 0;
    d |= 2u << 4;                       // D: s32
    d |= 0u << 7;                       // A: u8
    d |= 1u << 10;                      // B: s8
    d |= (uint32_t)(n >> 3) << 17;      // N
    d |= (uint32_t)(128 >> 4) << 24;    // M
    return d;
}

// The segments (group of four row blocks, range of pairs) of one stage that a CTA owns, in order.  The units of the
// stage, layer after layer and group-major inside a layer, are cut into equal contiguous shares: a CTA meets a
// segment boundary only where its share crosses from one group of row blocks into the next.
struct Seg {
    int li, rg, p0, p1, nseg, nrb;
};
// A CTA's share [u, u1) of the stage's units, cut at the group boundaries it contains.  The last segment's epilogue
// is the only one nothing hides, and a segment's epilogue cannot start before the previous one's has ended: when the
// share ends in a segment shorter than the one it starts with, the CTA walks its share backwards, so that the short
// segment's epilogue runs under the long one's streaming.  (Partial sums are added as integers: any order will do.)
struct SegIter {
    int stage, chunk, u, u1;
    bool backwards;
    struct Where { int li, rg, p, gstart, Np, R; };
    __device__ __forceinline__ Where locate(const Group &g, int unit) const {
        int li = 0;
        while (li + 1 < g.nlayers && unit >= g.layer[li + 1].st[stage].unit0) ++li;
        const Stage &S = g.layer[li].st[stage];
        const int local = unit - S.unit0;
        Where w;
        w.li = li; w.Np = S.Np; w.R = S.R;
        w.rg = local / S.Np;
        w.p = local - w.rg * S.Np;
        w.gstart = S.unit0 + w.rg * S.Np;
        return w;
    }
    __device__ __forceinline__ SegIter(const Group &g, int stage_, int cta, int) : stage(stage_) {
        chunk = g.chunk[stage];
        const int units = g.units[stage];
        u = min(cta * chunk, units);
        u1 = min(u + chunk, units);
        backwards = false;
        if (u < u1) {
            const Where a = locate(g, u), b = locate(g, u1 - 1);
            const int first_len = min(a.gstart + a.Np, u1) - u, last_len = u1 - max(b.gstart, u);
            backwards = last_len < first_len;
        }
    }
    __device__ __forceinline__ bool next(const Group &g, Seg &s) {
        if (u >= u1) return false;
        const Where w = locate(g, backwards ? u1 - 1 : u);
        const int lo = max(w.gstart, u), hi = min(w.gstart + w.Np, u1);     // the part of this group inside the share
        const int first = w.gstart / chunk, last = (w.gstart + w.Np - 1) / chunk;
        s.li = w.li; s.rg = w.rg; s.p0 = lo - w.gstart; s.p1 = hi - w.gstart; s.nseg = last - first + 1;
        s.nrb = min(kRBG, w.R - kRBG * w.rg);
        if (backwards) u1 = lo; else u = hi;
        return true;
    }
};

template <int LP> struct Cfg {
    static constexpr int NB = (3 * LP + 15) / 16 * 16;        // MMA N: three digits per mode, padded to a multiple of 16
    static constexpr int IMG = NB * 128;                      // bytes of one image
    static constexpr int NAG = 2;                             // A stages (32 columns) per row block: even and odd units
    static constexpr size_t SMEM = 1024 + (size_t)kImgSlots * IMG + (size_t)kSignSlots * 8192;
};

// named barrier of the four epilogue warps
__device__ __forceinline__ void aux_sync() { asm volatile("bar.sync 1, 128;\n" ::: "memory"); }

// N consecutive 16-bit envelope entries at p, two per register: vector loads when `vec` (p aligned to
// 2 N bytes, all N valid), otherwise the first `nvalid` by scalar loads and zeros for the rest.  No load
// depends on another.
template <int N> struct Row16 {
    uint32_t w[(N + 1) / 2];
    __device__ __forceinline__ uint16_t get(int t) const { return (uint16_t)(w[t >> 1] >> (16 * (t & 1))); }
};
template <int N>
__device__ __forceinline__ void load_row16(const uint16_t *p, bool vec, int nvalid, Row16<N> &out) {
    if (vec) {
        if constexpr (N >= 8) {
#pragma unroll
            for (int v = 0; v < N / 8; ++v) {
                const uint4 q = reinterpret_cast<const uint4 *>(p)[v];
                out.w[4 * v] = q.x; out.w[4 * v + 1] = q.y; out.w[4 * v + 2] = q.z; out.w[4 * v + 3] = q.w;
            }
        } else if constexpr (N == 4) {
            const uint2 q = *reinterpret_cast<const uint2 *>(p);
            out.w[0] = q.x; out.w[1] = q.y;
        } else if constexpr (N == 2) {
            out.w[0] = *reinterpret_cast<const uint32_t *>(p);
        } else {
            out.w[0] = p[0];
        }
    } else {
#pragma unroll
        for (int m = 0; m < (N + 1) / 2; ++m) {
            const uint32_t lo = 2 * m < nvalid ? p[2 * m] : 0u;
            const uint32_t hi = (2 * m + 1 < N && 2 * m + 1 < nvalid) ? p[2 * m + 1] : 0u;
            out.w[m] = lo | (hi << 16);
        }
    }
}
__device__ __forceinline__ float env16_to_float(uint16_t h, int env_dtype) {
    return env_dtype == MDBF_BF16 ? __uint_as_float((uint32_t)h << 16) : __half2float(__ushort_as_half(h));
}

// ------------------------------------------------------------------ image of one pair of K blocks
// Columns c = 128 p .. 128 p + 127 of the stage's input, scaled by V[c][t], as three signed digits of a
// fixed-point number; K position of column 32 w + 8 e + i inside the pair is 32 w + 4 i + e (byte e of
// the 32-bit word the expanders derive from (sign word w >> i)).  Thread layout: warp = group of LP / 4
// modes, lane = (w, i); a thread owns the four bytes e = 0..3 of one 32-bit word per (mode, digit).
// Split in two so that the loads of the immutable factors are in flight while the input is waited for.
template <int LP> struct ImgFactors {
    static constexpr int MT = LP >= 4 ? LP / 4 : 1;
    Row16<MT> v[4];
    float vmax[MT];
};
template <int LP>
__device__ __forceinline__ void load_image_factors(const LayerArgs &L, int s, int p, int atid, ImgFactors<LP> &f) {
    constexpr int MT = ImgFactors<LP>::MT;
    const Stage &S = L.st[s];
    const int mg = atid >> 5, lane = atid & 31, wq = lane >> 3, i = lane & 7;
    const bool active = mg * MT < LP;
    const uint16_t *V = reinterpret_cast<const uint16_t *>(S.V);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int c = 128 * p + 32 * wq + 8 * e + i;
        const bool ok = active && c < S.cols;
        const int nvalid = ok ? max(0, min(MT, L.l - mg * MT)) : 0;
        load_row16<MT>(V + (size_t)c * L.l + mg * MT, ok && L.l == LP, nvalid, f.v[e]);
    }
#pragma unroll
    for (int m = 0; m < MT; ++m) f.vmax[m] = active ? S.vmax[mg * MT + m] : 0.f;
}
// the four input values of this thread's columns (x for stage B, z for stage A)
__device__ __forceinline__ void load_image_inputs(const LayerArgs &L, int s, int p, int atid, float (&in)[4]) {
    const Stage &S = L.st[s];
    const int lane = atid & 31, wq = lane >> 3, i = lane & 7;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int c = 128 * p + 32 * wq + 8 * e + i;
        const int cc = c < S.cols ? c : 0;
        const float v = s == 0 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(L.x)[cc]) : __ldcg(L.z + cc);
        in[e] = c < S.cols ? v : 0.f;
    }
}
// tile: where the image goes (the layer's image buffer in global memory, or an image slot of this CTA's
// shared memory); cs_out: where the pair's column sums go ([32] ints), or null
template <int LP>
__device__ __forceinline__ void build_image(const LayerArgs &L, int s, const float (&in)[4], float amax, int atid, const ImgFactors<LP> &f,
                                            int8_t *tile, int *cs_out) {
    constexpr int MT = ImgFactors<LP>::MT;
    const int mg = atid >> 5, lane = atid & 31, wq = lane >> 3, i = lane & 7;
    int csum[MT];                                 // |sum| <= 128 * 2^20
#pragma unroll
    for (int m = 0; m < MT; ++m) csum[m] = 0;
    if (mg * MT >= LP) return;                    // whole warps only (LP < 4)
    float inv[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        const float bound = amax * f.vmax[m];
        inv[m] = bound > 0.f ? kQmax / bound : 0.f;
    }
    uint32_t w[MT][3];
#pragma unroll
    for (int m = 0; m < MT; ++m) w[m][0] = w[m][1] = w[m][2] = 0u;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            const float v = env16_to_float(f.v[e].get(m), L.env_dtype);
            const int q = __float2int_rn(in[e] * v * inv[m]);
            csum[m] += q;
            const int q2 = (q + 8192) >> 14;
            const int r = q - (q2 << 14);
            const int q1 = (r + 64) >> 7;
            const int q0 = r - (q1 << 7);
            w[m][0] |= (uint32_t)(q0 & 0xFF) << (8 * e);
            w[m][1] |= (uint32_t)(q1 & 0xFF) << (8 * e);
            w[m][2] |= (uint32_t)(q2 & 0xFF) << (8 * e);
        }
    }
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int j = 0; j < 3; ++j) {
            const int n = j * LP + mg * MT + m;
            const int off = n * 128 + (((2 * wq + (i >> 2)) ^ (n & 7)) << 4) + ((i & 3) << 2);
            *reinterpret_cast<uint32_t *>(tile + off) = w[m][j];
        }
    if (!cs_out) return;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        int v = csum[m];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) cs_out[mg * MT + m] = v;
    }
}

// max |x| over a bf16 vector by every thread of the CTA (unrolled: several loads per thread in flight)
__device__ __forceinline__ float amax_bf16_block(const void *x, int n, float *redw) {
    const __nv_bfloat16 *xp = reinterpret_cast<const __nv_bfloat16 *>(x);
    const int tid = threadIdx.x, nthr = blockDim.x;
    float m = 0.f;
    if ((reinterpret_cast<uintptr_t>(x) & 15u) == 0) {
        const int n8 = n >> 3;
#pragma unroll 8
        for (int v8 = tid; v8 < n8; v8 += nthr) {
            const uint4 q = reinterpret_cast<const uint4 *>(x)[v8];
            const uint32_t ws[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                m = fmaxf(m, fabsf(__uint_as_float(ws[e] << 16)));
                m = fmaxf(m, fabsf(__uint_as_float(ws[e] & 0xFFFF0000u)));
            }
        }
        for (int c = (n8 << 3) + tid; c < n; c += nthr) m = fmaxf(m, fabsf(__bfloat162float(xp[c])));
    } else {
#pragma unroll 8
        for (int c = tid; c < n; c += nthr) m = fmaxf(m, fabsf(__bfloat162float(xp[c])));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((tid & 31) == 0) redw[tid >> 5] = m;
    __syncthreads();
    m = redw[0];
    for (int w = 1; w < (nthr >> 5); ++w) m = fmaxf(m, redw[w]);
    return m;
}

// max |z| over an fp32 vector (the intermediate, written by the previous kernel) by every thread of the CTA
__device__ __forceinline__ float amax_f32_block(const float *z, int n, float *redw) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    float m = 0.f;
    const int n4 = n >> 2;                        // cudaMalloc'ed buffer: 16-byte aligned
#pragma unroll 8
    for (int v4 = tid; v4 < n4; v4 += nthr) {
        const float4 q = __ldcg(reinterpret_cast<const float4 *>(z) + v4);
        m = fmaxf(fmaxf(m, fabsf(q.x)), fmaxf(fabsf(q.y), fmaxf(fabsf(q.z), fabsf(q.w))));
    }
    for (int c = (n4 << 2) + tid; c < n; c += nthr) m = fmaxf(m, fabsf(__ldcg(z + c)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((tid & 31) == 0) redw[tid >> 5] = m;
    __syncthreads();
    m = redw[0];
    for (int w = 1; w < (nthr >> 5); ++w) m = fmaxf(m, redw[w]);
    return m;
}

// ------------------------------------------------------------------------ image kernel
// One CTA per pair of K blocks of every layer of the launch (stage s): the operand images of the stage (four pairs
// per CTA measured 2-9 % slower on the 70B-class block).
// Every CTA makes its own pass over the stage's input (x, or an intermediate z that another kernel produced) for its
// largest magnitude: a few KB out of L2, cheaper than a reduction across CTAs.  The stage kernel of this file leaves
// max |z| behind (one atomic maximum per warp of finished rows), so stage A after it skips the pass.
template <int LP>
__global__ void __launch_bounds__(kImgThreads) t1_image_kernel(const __grid_constant__ Group g, const int s, const int have_amax) {
    constexpr int IMG = Cfg<LP>::IMG;
    __shared__ float redw[kImgThreads / 32];
    const int tid = threadIdx.x;
    const int m = blockIdx.x;
    int li = 0;
    while (li + 1 < g.nlayers && m >= g.layer[li + 1].st[s].item0) ++li;
    const LayerArgs &L = g.layer[li];
    const int atid = tid & 127;
    const int p = m - L.st[s].item0;
    const bool builds = tid < 128;
    tm::pdl_launch_dependents();
    ImgFactors<LP> fac;
    if (builds) load_image_factors<LP>(L, s, p, atid, fac);      // immutable: in flight while the previous kernel drains
    tm::pdl_wait();
    float in[4] = {0.f, 0.f, 0.f, 0.f};
    if (builds) load_image_inputs(L, s, p, atid, in);            // requested before the pass below: one round trip, not two
    float amax;
    if (have_amax) {                                             // stage A after this file's stage B: its epilogue left max |z|
        amax = __uint_as_float(__ldcg(L.sync + kSyAmax + 1));
    } else {
        amax = s == 0 ? amax_bf16_block(L.x, L.st[0].cols, redw) : amax_f32_block(L.z, L.st[1].cols, redw);
        if (p == 0 && atid == 0) L.sync[kSyAmax + s] = __float_as_uint(amax);
    }
    if (s == 0 && p == 0 && atid == 0) L.sync[kSyAmax + 1] = 0u; // stage B's epilogue takes the maximum into it
    if (builds) build_image<LP>(L, s, in, amax, atid, fac, L.st[s].img + (size_t)p * IMG, L.st[s].colsum + p * 32);
}

// ------------------------------------------------------------------------ stage kernel
template <int LP>
__global__ void __launch_bounds__(kThreads, 1) t1_stage_kernel(const __grid_constant__ Group g, const int s) {
    using namespace tm;
    constexpr int NB = Cfg<LP>::NB;
    constexpr int IMG = Cfg<LP>::IMG;
    constexpr int NAG = Cfg<LP>::NAG;
    constexpr int NSQ = kSignSlots, NIM = kImgSlots;
    constexpr int TMEM_COLS = 512;
    constexpr int W_AUX = 16, W_ISS = 20, W_SLOAD = W_ISS + kIssuers;   // then the image loader warp
    // barriers: s_full[NSQ] s_empty[NSQ] i_full[NIM] i_empty[NIM] a_full[4][NAG] acc_full acc_empty
    constexpr int B_SF = 0, B_SE = NSQ, B_IF = 2 * NSQ, B_IE = 2 * NSQ + NIM, B_AF = 2 * NSQ + 2 * NIM,
                  B_ACF = B_AF + 4 * NAG, B_ACE = B_ACF + 1, NBARS = B_ACE + 1;

    extern __shared__ unsigned char t1_smem_raw[];
    __shared__ __align__(8) uint64_t bars[NBARS];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;
    __shared__ unsigned long long cs_s[32];
    volatile int *abort_flag = &abort_flag_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;
    const uint32_t smem_base = (smem_u32(t1_smem_raw) + 1023u) & ~1023u;
    unsigned char *smem_gen = t1_smem_raw + (smem_base - smem_u32(t1_smem_raw));
    const uint32_t off_s = (uint32_t)(NIM * IMG);                // sign ring after the image ring

    const uint32_t bar0 = smem_u32(&bars[0]);
    const uint32_t s_full = bar0 + 8 * B_SF, s_empty = bar0 + 8 * B_SE, i_full = bar0 + 8 * B_IF, i_empty = bar0 + 8 * B_IE,
                   a_full = bar0 + 8 * B_AF, acc_full = bar0 + 8 * B_ACF, acc_empty = bar0 + 8 * B_ACE;
    int32_t *status0 = g.layer[0].status;

    if (tid < NBARS) {
        uint32_t count = 1u;                                     // s_full, i_full (expect_tx)
        if (tid >= B_SE && tid < B_IF) count = 16u;              // s_empty: every expander warp
        else if (tid >= B_IE && tid < B_AF) count = 4u;          // i_empty: every issuer (commit)
        else if (tid >= B_AF && tid < B_ACF) count = 4u;         // a_full: the four warps of the group
        else if (tid == B_ACF) count = (uint32_t)kIssuers;       // acc_full: every issuer
        else if (tid == B_ACE) count = 4u;                       // acc_empty: the four epilogue warps
        mbar_init(bar0 + 8 * tid, count);
    }
    if (tid == 0) abort_flag_s = 0;
    fence_barrier_init();
    if (warp == W_ISS) {
        tmem_alloc(smem_u32(&tmem_base_slot), (uint32_t)TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    const uint32_t tmem_a0 = tmem + (uint32_t)(4 * NB);         // A stages: [row block j][NAG][32 columns]

    pdl_launch_dependents();

    if (warp < W_AUX) {
        // ===================================== expanders =====================================
        const int grp = warp >> 2;                               // row block of the unit
        const int row_l = (warp & 3) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        bool alive = true;
        int qn = 0;                                              // units this CTA has walked
        int prev_as = -1;                                        // A stage whose stores are still to be published
        SegIter it(g, s, cta, (int)gridDim.x);
        Seg sg;
        while (alive && it.next(g, sg)) {
            const bool valid = grp < sg.nrb;
            for (int p = sg.p0; p < sg.p1; ++p, ++qn) {
                const int rs = qn % NSQ;
                alive = bwait(s_full + 8 * rs, (uint32_t)(qn / NSQ) & 1u, abort_flag, status0);
                if (!alive) break;
                uint2 w0 = make_uint2(0u, 0u), w1 = w0;
                if (valid) {
                    const unsigned char *sw = smem_gen + off_s + rs * 8192 + grp * 2048 + row_l * 8;
                    w0 = *reinterpret_cast<const uint2 *>(sw);
                    w1 = *reinterpret_cast<const uint2 *>(sw + 1024);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty + 8 * rs);
                if (prev_as >= 0) {                              // publish the previous unit: its stores had a unit's time to land
                    tmem_st_wait();                              // (before the validity test: the row block may not exist in this unit)
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(a_full + 8 * (grp * NAG + prev_as));
                    prev_as = -1;
                }
                if (!valid) continue;
                // the 32 operand words of this row are finished in registers before the A stage is claimed (the MMAs of
                // the unit that used the stage two units ago may still run): only the stores follow the wait
                const uint32_t ws[4] = {w0.x, w0.y, w1.x, w1.y};
                uint32_t v[32];                                  // sign word q -> TMEM columns 8q .. 8q+7
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[8 * q + i] = (ws[q] * g.shl_mul[i]) & 0x80808080u;   // bit 8e + i -> top bit of byte e
                // A stage qn % NAG: whatever this row block last put there was consumed by unit qn - NAG at the latest, and
                // every issuer releases a unit's image with a commit, i.e. after all its earlier MMAs have retired: one
                // commit per unit and issuer serves both rings.
                const int as = qn % NAG;
                if (qn >= NAG) {
                    const int qp = qn - NAG;
                    alive = bwait(i_empty + 8 * (qp % NIM), (uint32_t)(qp / NIM) & 1u, abort_flag, status0);
                    if (!alive) break;
                }
                tc_fence_after();
                const uint32_t a_col = tmem_a0 + lane_base + (uint32_t)((grp * NAG + as) * 32);
                tmem_st32(a_col, v);                             // one store of the whole row: a tcgen05.st holds the warp for ~140 clocks whatever its width
                prev_as = as;
            }
        }
        if (prev_as >= 0) {
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (alive && lane == 0) mbar_arrive(a_full + 8 * (grp * NAG + prev_as));
        }
    } else if (warp < W_ISS) {
        // ============================ epilogue warps: contraction with U, row finalisation ============================
        const int atid = tid - W_AUX * 32;                       // 0 .. 127 = row of the tile = TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        bool alive = true;
        int nseg_done = 0;                                       // segments this CTA has finished: phase of the accumulator barriers
        // Every MMA accumulates (two issuers share a row block's accumulator, so none of them can be "the first"): the
        // accumulators are cleared here, before the first segment and after each read.
        {
            const uint32_t zero[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
            for (int c8 = 0; c8 < 4 * NB / 8; ++c8) tmem_st8(tmem + lane_base + (uint32_t)(c8 * 8), zero);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty);
        }
        SegIter it(g, s, cta, (int)gridDim.x);
        Seg sg;
        while (alive && it.next(g, sg)) {
            const LayerArgs &L = g.layer[sg.li];
            const Stage &S = L.st[s];
            // U rows of this thread's row in the (up to) four row blocks and the mode scales: immutable, in flight during the MMAs
            Row16<LP> urow[kRBG];
#pragma unroll
            for (int j = 0; j < kRBG; ++j) {
                const int grow = (sg.rg * kRBG + j) * 128 + atid;
                const bool ok = j < sg.nrb && grow < S.rows;
                load_row16<LP>(reinterpret_cast<const uint16_t *>(S.U) + (size_t)grow * L.l, ok && L.l == LP, ok ? L.l : 0, urow[j]);
            }
            float scale[LP];
#pragma unroll
            for (int t = 0; t < LP; ++t) scale[t] = S.vmax[t];
            if (nseg_done == 0) pdl_wait();                      // what follows is the previous kernel's output
            // column sums of q over the pairs of this segment: warp w takes every fourth pair, lane = mode
            {
                aux_sync();                                      // cs_s may still be read from the previous segment
                if (atid < 32) cs_s[atid] = 0ull;
                aux_sync();
                long long v = 0;
                if ((atid & 31) < LP)
                    for (int p = sg.p0 + (atid >> 5); p < sg.p1; p += 4) v += __ldcg(S.colsum + p * 32 + (atid & 31));
                if ((atid & 31) < LP) atomicAdd(&cs_s[atid & 31], (unsigned long long)v);
                aux_sync();
            }
            const float am = __uint_as_float(__ldcg(L.sync + kSyAmax + s)) * (1.f / kQmax);
#pragma unroll
            for (int t = 0; t < LP; ++t) scale[t] *= am;
            mbar_wait(acc_full, (uint32_t)nseg_done & 1u, abort_flag, L.status);
            aux_sync();                                          // one decision for the whole group
            if (*abort_flag) { alive = false; break; }
            tc_fence_after();
            // First only what needs the accumulators: per row block the three digits of every mode combined into one float,
            // f[j][t] = -2 * sum_c b q[c][t] (the A bytes are 128 b: -2 * 128^digit / 128), and the accumulator cleared; then
            // the issuers may start the next segment while the contraction with U and the hand-over run here.
            float f[kRBG][LP];
#pragma unroll
            for (int j = 0; j < kRBG; ++j) {
#pragma unroll
                for (int t = 0; t < LP; ++t) f[j][t] = 0.f;
                if (j < sg.nrb) {
#pragma unroll
                    for (int c16 = 0; c16 < NB / 16; ++c16) {
                        uint32_t d[16];
                        tmem_ld16(tmem + lane_base + (uint32_t)(j * NB + c16 * 16), d);
                        tmem_ld_wait();
                        const uint32_t zero[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
                        tmem_st8(tmem + lane_base + (uint32_t)(j * NB + c16 * 16), zero);
                        tmem_st8(tmem + lane_base + (uint32_t)(j * NB + c16 * 16 + 8), zero);
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const int col = c16 * 16 + e;
                            if (col < 3 * LP) {
                                const int jd = col / LP, t = col % LP;
                                const float wgt = jd == 0 ? -0.015625f : jd == 1 ? -2.f : -256.f;
                                f[j][t] = fmaf(wgt, (float)(int)d[e], f[j][t]);
                            }
                        }
                    }
                }
            }
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty);               // read and cleared: the issuers may start the next segment
            ++nseg_done;

            float part[kRBG];
#pragma unroll
            for (int j = 0; j < kRBG; ++j) {
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int t = 0; t < LP; ++t)                     // contraction with U; + sum_c q over the segment's pairs (S = 1 - 2 b)
                    acc[t & 3] = fmaf(env16_to_float(urow[j].get(t), L.env_dtype) * scale[t], f[j][t] + (float)(long long)cs_s[t], acc[t & 3]);
                part[j] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
            }

            // A group split over several CTAs.  Every segment adds, per row, its partial output as a fixed-point number in
            // the upper 56 bits of the row's 64-bit accumulator and 1 in the lower 8 (integer addition: the order of
            // arrival does not matter); the thread whose addition completes the count has the row's sum in hand, clears
            // the accumulator and finalises the row.  The exponent of a row's fixed point follows from a bound on its
            // output that every segment computes alike: |out| < sum_t |u_t delta_t| * cols * 2^22.
            bool fin[kRBG];
#pragma unroll
            for (int j = 0; j < kRBG; ++j) {
                const int grow = (sg.rg * kRBG + j) * 128 + atid;
                fin[j] = j < sg.nrb && grow < S.rows;
            }
            if (sg.nseg > 1) {
                int fexp[kRBG];
                unsigned long long mine[kRBG], old[kRBG];
#pragma unroll
                for (int j = 0; j < kRBG; ++j) {
                    float sabs = 0.f;
#pragma unroll
                    for (int t = 0; t < LP; ++t) sabs += fabsf(env16_to_float(urow[j].get(t), L.env_dtype) * scale[t]);
                    const float bound = sabs * (float)(S.Np * 128) * 4194304.f;
                    fexp[j] = max(-60, min(100, (int)((__float_as_uint(bound) >> 23) & 0xFFu) - 126));   // bound < 2^fexp (clamped: powers of two below stay normal floats)
                    mine[j] = ((unsigned long long)__float2ll_rn(part[j] * 67108864.f * __uint_as_float((uint32_t)(127 + 27 - fexp[j]) << 23)) << 8) + 1ull;
                    old[j] = 0ull;
                }
#pragma unroll
                for (int j = 0; j < kRBG; ++j)
                    if (fin[j] && store_in_bounds((size_t)((sg.rg * kRBG + j) * 128 + atid), (size_t)S.R * 128, L.status))
                        old[j] = atomicAdd(S.acc64 + (sg.rg * kRBG + j) * 128 + atid, mine[j]);
                    else fin[j] = false;
#pragma unroll
                for (int j = 0; j < kRBG; ++j)
                    if (fin[j]) {
                        fin[j] = (int)(old[j] & 0xFFull) + 1 == sg.nseg;
                        if (fin[j]) {
                            __stcg(S.acc64 + (sg.rg * kRBG + j) * 128 + atid, 0ull);
                            const long long tot = (long long)(old[j] + mine[j]) >> 8;
                            part[j] = (float)tot * 1.4901161193847656e-08f * __uint_as_float((uint32_t)(127 - 27 + fexp[j]) << 23);   // 2^-26 * 2^(fexp - 27)
                        }
                    }
            }
            if (s == 0) {
                float zmax = 0.f;
#pragma unroll
                for (int j = 0; j < kRBG; ++j)
                    if (fin[j] && store_in_bounds((size_t)((sg.rg * kRBG + j) * 128 + atid), (size_t)S.rows, L.status)) {
                        L.z[(sg.rg * kRBG + j) * 128 + atid] = part[j];
                        zmax = fmaxf(zmax, fabsf(part[j]));
                    }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, o));
                if (lane == 0 && zmax > 0.f) atomicMax(L.sync + kSyAmax + 1, __float_as_uint(zmax));   // non-negative floats order like their bits
            } else {
#pragma unroll
                for (int j = 0; j < kRBG; ++j)
                    if (fin[j]) {
                        const int grow = (sg.rg * kRBG + j) * 128 + atid;
                        if (!store_in_bounds((size_t)grow, (size_t)S.rows, L.status)) continue;
                        if (L.out_mode == 0) reinterpret_cast<__nv_bfloat16 *>(L.y)[grow] = __float2bfloat16_rn(part[j]);
                        else if (L.out_mode == 1) reinterpret_cast<float *>(L.y)[grow] = part[j];
                        else reinterpret_cast<float *>(L.y)[grow] += part[j];
                    }
            }
        }
    } else if (warp < W_SLOAD) {
        // ==================================== MMA issuers ====================================
        // Two issuers per row block of the unit, one for the even and one for the odd units (= A stage 0 / 1): while one
        // of them is between units, the other keeps the tensor pipe fed.  Both accumulate into the row block's
        // accumulator (integer addition: the order does not matter).
        const int k = (warp - W_ISS) & 3;                        // row block of the unit
        const int par = (warp - W_ISS) >> 2;                     // units this issuer takes: qn % 2 == par
        const uint32_t idesc = make_idesc_i8(NB);
        const uint32_t d_tmem = tmem + (uint32_t)(k * NB);
        bool alive = true;
        int qn = 0, nseg_done = 0;
        uint32_t ause = 0u;                                      // uses of this issuer's A stage so far
        SegIter it(g, s, cta, (int)gridDim.x);
        Seg sg;
        while (alive && it.next(g, sg)) {
            const bool valid = k < sg.nrb;
            alive = bwait(acc_empty, (uint32_t)nseg_done & 1u, abort_flag, status0);   // accumulators read and cleared
            if (!alive) break;
            int issued = 0;
            for (int p = sg.p0; p < sg.p1 && alive; ++p, ++qn) {
                if ((qn & 1) != par) continue;
                const int is = qn % NIM;
                alive = bwait(i_full + 8 * is, (uint32_t)(qn / NIM) & 1u, abort_flag, status0);
                if (!alive) break;
                if (!valid) {                                    // no such row block: only release the image (after this issuer's earlier MMAs)
                    if (lane == 0) umma_commit(i_empty + 8 * is);
                    __syncwarp();
                    continue;
                }
                alive = bwait(a_full + 8 * (k * NAG + par), ause & 1u, abort_flag, status0);
                if (!alive) break;
                tc_fence_after();
                if (lane == 0) {
                    const uint64_t bdesc = make_smem_desc(smem_base + (uint32_t)(is * IMG));
                    const uint32_t a_t = tmem_a0 + (uint32_t)((k * NAG + par) * 32);
#pragma unroll
                    for (int q = 0; q < 4; ++q)                  // 32 K positions (bytes) per MMA
                        umma_ts_i8(d_tmem, a_t + (uint32_t)(8 * q), bdesc + (uint64_t)(2 * q), idesc, 1u);
                    umma_commit(i_empty + 8 * is);               // one of the four releases of the image; with all four the A stages of the unit are free too
                }
                __syncwarp();
                ++issued;
                ++ause;
            }
            if (lane == 0) {
                if (alive && issued > 0) umma_commit(acc_full);  // arrives when this issuer's MMAs have retired
                else mbar_arrive(acc_full);
            }
            __syncwarp();
            ++nseg_done;
        }
    } else if (warp == W_SLOAD) {
        // ================================= sign-word loader ==================================
        // Lane l owns ring slot l: it waits for the slot, then issues the (up to) four bulk copies of its unit.  Sign
        // words are immutable: no need to wait for the previous kernel.
        if (lane < NSQ) {
            bool alive = true;
            int qn = 0;
            SegIter it(g, s, cta, (int)gridDim.x);
            Seg sg;
            while (alive && it.next(g, sg)) {
                const Stage &S = g.layer[sg.li].st[s];
                const size_t rb_stride = (size_t)S.kb_pad * 128;
                const uint2 *src = S.wk2 + ((size_t)sg.rg * kRBG * S.kb_pad + 2 * (size_t)sg.p0) * 128;
                for (int p = sg.p0; p < sg.p1; ++p, ++qn, src += 256) {
                    if (qn % NSQ != lane) continue;
                    alive = bwait(s_empty + 8 * lane, ((uint32_t)(qn / NSQ) & 1u) ^ 1u, abort_flag, status0);
                    if (!alive) break;
                    mbar_arrive_expect_tx(s_full + 8 * lane, 2048u * (uint32_t)sg.nrb);
                    for (int j = 0; j < sg.nrb; ++j)
                        bulk_load(smem_base + off_s + (uint32_t)(lane * 8192 + j * 2048), src + j * rb_stride, 2048u, s_full + 8 * lane);
                }
            }
            if (!alive) drain_delay();
        }
        __syncwarp();
    } else {
        // =================================== image loader ====================================
        // Lane l owns ring slot l.  The images are the previous kernel's output.
        if (lane < NIM) {
            bool alive = true;
            int qn = 0;
            pdl_wait();
            fence_proxy_async_all();                             // written through the generic proxy, read by bulk copies
            SegIter it(g, s, cta, (int)gridDim.x);
            Seg sg;
            while (alive && it.next(g, sg)) {
                const Stage &S = g.layer[sg.li].st[s];
                for (int p = sg.p0; p < sg.p1 && alive; ++p, ++qn) {
                    if (qn % NIM != lane) continue;
                    alive = bwait(i_empty + 8 * lane, ((uint32_t)(qn / NIM) & 1u) ^ 1u, abort_flag, status0);
                    if (!alive) break;
                    mbar_arrive_expect_tx(i_full + 8 * lane, (uint32_t)IMG);
                    bulk_load(smem_base + (uint32_t)(lane * IMG), S.img + (size_t)p * IMG, (uint32_t)IMG, i_full + 8 * lane);
                }
            }
            if (!alive) drain_delay();
        }
        __syncwarp();
    }

    // ------------------------------ leave ------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == W_ISS) tmem_dealloc(tmem, (uint32_t)TMEM_COLS);
    if (tid == 0) {
        pdl_wait();                                              // a kernel that ends has seen its predecessor end
        if (abort_flag_s)
            for (int li = 0; li < g.nlayers; ++li) atomicExch(g.layer[li].status, (int32_t)MDBF_ERR_TIMEOUT);
    }
}

// max_c |V[c][t]| per mode (pack time): one block per mode
__global__ void vmax_kernel(const void *__restrict__ V, int cols, int l, int env_dtype, float *__restrict__ out) {
    __shared__ float red[8];
    const int t = blockIdx.x;
    float m = 0.f;
    if (t < l)
        for (int c = threadIdx.x; c < cols; c += blockDim.x) m = fmaxf(m, fabsf(env_load(V, (size_t)c * l + t, env_dtype)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) m = fmaxf(m, red[w]);
        out[t] = m;
    }
}

}  // namespace t1

// ---------------------------------------------------------------------------- host side
static int t1_cta_count() {
    static int per_device[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!per_device[dev]) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        per_device[dev] = sms;
    }
    return per_device[dev];
}

// Scratch and pack-time constants of the one-token kernel (16-bit envelopes, l <= 32).
mdbf_status_t t1_prepare(Layer &L, cudaStream_t st) {
    const mdbf_desc_t &d = L.d;
    const int C = t1_cta_count();
    if (C <= 0) { set_error("mdbf_pack: cannot query the SM count"); return MDBF_ERR_CUDA; }
    T1Buffers &b = L.t1;
    const int NB = (3 * L.LP + 15) / 16 * 16;
    b.NB = NB;
    b.ctas = C;
    b.R[0] = L.rpB / 128; b.Np[0] = L.kbpB / 2;
    b.R[1] = L.rpA / 128; b.Np[1] = L.kbpA / 2;
    for (int s = 0; s < 2; ++s) b.RG[s] = ceil_div(b.R[s], t1::kRBG);
    MDBF_CUDA(dev_malloc(&b.vmax, 64 * sizeof(float)));
    MDBF_CUDA(dev_malloc(&b.sync, (size_t)t1::kSyWords * 4));
    MDBF_CUDA(cudaMemsetAsync(b.sync, 0, (size_t)t1::kSyWords * 4, st));
    for (int s = 0; s < 2; ++s) {
        MDBF_CUDA(dev_malloc(&b.img[s], (size_t)b.Np[s] * NB * 128));
        MDBF_CUDA(cudaMemsetAsync(b.img[s], 0, (size_t)b.Np[s] * NB * 128, st));      // the padding rows stay zero
        MDBF_CUDA(dev_malloc(&b.colsum[s], (size_t)b.Np[s] * 32 * sizeof(int)));
        MDBF_CUDA(cudaMemsetAsync(b.colsum[s], 0, (size_t)b.Np[s] * 32 * sizeof(int), st));
        MDBF_CUDA(dev_malloc(&b.acc64[s], (size_t)b.R[s] * 128 * sizeof(unsigned long long)));
        MDBF_CUDA(cudaMemsetAsync(b.acc64[s], 0, (size_t)b.R[s] * 128 * sizeof(unsigned long long), st));
    }
    MDBF_CUDA(cudaMemsetAsync(b.vmax, 0, 64 * sizeof(float), st));
    t1::vmax_kernel<<<L.LP, 256, 0, st>>>(L.VB, d.d_in, d.l, d.env_dtype, b.vmax);
    t1::vmax_kernel<<<L.LP, 256, 0, st>>>(L.VA, d.k, d.l, d.env_dtype, b.vmax + 32);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

void t1_release(Layer &L) {
    T1Buffers &b = L.t1;
    void *ptrs[] = {b.vmax, b.sync, b.img[0], b.img[1], b.colsum[0], b.colsum[1], b.acc64[0], b.acc64[1]};
    for (void *p : ptrs)
        if (p) cudaFree(p);
    b = T1Buffers{};
}

bool t1_supports(const Layer &L) { return L.t1.sync != nullptr && L.wk2A != nullptr && L.LP <= 16 && L.d.d_in <= (1 << 17) && L.d.k <= (1 << 17); }

template <typename Kern, typename... Args>
static mdbf_status_t t1_launch_one(Kern kern, int grid, int block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    MDBF_CUDA(cudaLaunchKernelEx(&cfg, kern, args...));
    return MDBF_OK;
}

template <int LP>
static mdbf_status_t t1_launch(const t1::Group &grp, int ctas, cudaStream_t st, int stages) {
    auto stage_kern = t1::t1_stage_kernel<LP>;
    auto image_kern = t1::t1_image_kernel<LP>;
    const size_t smem = t1::Cfg<LP>::SMEM;
    static PerDeviceOnce once;
    if (once.first()) MDBF_CUDA(cudaFuncSetAttribute(stage_kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    for (int s = 0; s < 2; ++s) {
        if (!(stages >> s & 1)) continue;
        // stage A right after this file's stage B: max |z| is already there
        mdbf_status_t rc = t1_launch_one(image_kern, grp.items[s], t1::kImgThreads, 0, st, grp, s, (int)(s == 1 && stages == 3));
        if (rc) return rc;
        rc = t1_launch_one(stage_kern, ctas, t1::kThreads, smem, st, grp, s);
        if (rc) return rc;
    }
    return MDBF_OK;
}

// One or both stages of n <= 8 layers, two launches per stage (image kernel, stage kernel).  xs[i] / ys[i]: bf16
// input and output of layer i — layers may share an input; the intermediate z of a layer is its handle's fp32
// buffer, whoever writes or reads it.  stages: bit 0 = stage B (x -> z), bit 1 = stage A (z -> y).  All layers have
// the same LP and were prepared by t1_prepare.
mdbf_status_t launch_forward_t1_group(Layer *const *Ls, int n, const void *const *xs, void *const *ys, cudaStream_t st, int stages) {
    if (n < 1 || n > t1::kMaxLayers) { set_error("one-token kernel: %d layers in one launch (at most %d)", n, t1::kMaxLayers); return MDBF_ERR_SHAPE; }
    t1::Group grp = {};
    grp.nlayers = n;
    for (int i = 0; i < 8; ++i) grp.shl_mul[i] = 128u >> i;
    const int C = Ls[0]->t1.ctas;
    for (int i = 0; i < n; ++i) {
        Layer &L = *Ls[i];
        if (!t1_supports(L) || L.LP != Ls[0]->LP || L.t1.ctas != C) { set_error("one-token kernel: layer %d was not prepared for it", i); return MDBF_ERR_INVALID_ARG; }
        t1::LayerArgs &a = grp.layer[i];
        const T1Buffers &b = L.t1;
        for (int s = 0; s < 2; ++s) {
            t1::Stage &S = a.st[s];
            S.wk2 = s ? L.wk2A : L.wk2B;
            S.V = s ? L.VA : L.VB;
            S.U = s ? L.UA : L.UB;
            S.vmax = b.vmax + 32 * s;
            S.img = b.img[s];
            S.colsum = b.colsum[s];
            S.acc64 = b.acc64[s];
            S.rows = s ? L.d.d_out : L.d.k;
            S.cols = s ? L.d.k : L.d.d_in;
            S.R = b.R[s]; S.RG = b.RG[s]; S.Np = b.Np[s];
            S.kb_pad = s ? L.kbpA : L.kbpB;
            S.unit0 = grp.units[s];
            S.item0 = grp.items[s];
            grp.units[s] += S.RG * S.Np;
            grp.items[s] += S.Np;
        }
        a.x = xs[i];
        a.z = L.zsum;
        a.y = ys[i];
        a.sync = b.sync;
        a.status = L.status;
        a.l = L.d.l; a.env_dtype = L.d.env_dtype; a.out_mode = L.out_mode;
    }
    for (int s = 0; s < 2; ++s) grp.chunk[s] = ceil_div(grp.units[s], C);
    switch (Ls[0]->LP) {
        case 1: return t1_launch<1>(grp, C, st, stages);
        case 2: return t1_launch<2>(grp, C, st, stages);
        case 4: return t1_launch<4>(grp, C, st, stages);
        case 8: return t1_launch<8>(grp, C, st, stages);
        case 16: return t1_launch<16>(grp, C, st, stages);
        default:
            set_error("one-token integer kernel: l <= 16 (got %d)", Ls[0]->d.l);
            return MDBF_ERR_SHAPE;
    }
}

}  // namespace mdbf
