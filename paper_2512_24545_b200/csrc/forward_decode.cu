// Small-T ("decode") path of the MDBF forward: T <= 4 tokens, l <= 32.
//
// One stage computes, for the rows r of a packed sign matrix S (rows x cols),
//
//     out[tau][r] = sum_t U[r][t] * sum_c S[r][c] * V[c][t] * in[tau][c]
//
// (sum_t D_{u_t} S D_{v_t} applied to `in`, Eq. me-dbf-expand).  Stage B runs it
// with (S_B, V_B, U_B) on x and leaves split-K partial sums of z in scratch;
// stage A runs it with (S_A, V_A, U_A) on z and writes y (Eq.
// DBF-inference-form, column convention).
//
// Mapping to the warp-level tensor-core MMA (m16n8k16, bf16 in, fp32 out), per
// token:  A[r][c] = S[r][c] * in[c]  (the activation with the packed bit XOR-ed
// into its bf16 sign bit — add/sub only, no multiply by the sign),
// B[c][t] = V[c][t] (bf16), D[r][t] accumulates in fp32; the mode contraction
// with U is a quad shuffle reduction in the epilogue.  The sign matrix and V
// are streamed once and shared by the l envelope modes and the tokens.
//
// Data movement: sign tiles are read with one 128-bit load per lane from the
// tiled copy (a warp reads 512 contiguous bytes); V arrives in B-fragment
// order through cp.async into a double-buffered shared-memory ring; both are
// immutable weights and are requested BEFORE the programmatic-dependent-launch
// wait, so with back-to-back launches the next layer's weights stream in while
// the previous kernel drains.  Activations are staged after the wait.
#include <cstdlib>

#include "common.cuh"

namespace mdbf {

constexpr int DEC_THREADS = 256;
constexpr int DEC_WARPS = 8;
constexpr int DEC_CT = 8;          // 128-column sign tiles per shared-memory chunk of V
constexpr int DEC_MAX_TPW = 4;     // sign tiles a warp owns per chunk (= WR)

struct StageArgs {
    const uint4 *tiled;   // sign tiles, [rtiles][ktiles][32 lanes]
    int rtiles, ktiles;
    const uint2 *vfrag;   // V in B-fragment order, [ktiles][8 steps][NT][32 lanes]
    const void *U;        // [rows][l], env_dtype
    int env_dtype, l;
    int rows, cols;
    const __nv_bfloat16 *x;   // stage B input  [T][cols]
    const float *zin;         // stage A input  [nsplit_in][T][cols] partial sums
    int nsplit_in;
    size_t zin_stride;
    float *zout;              // stage B output [gridDim.y][T][rows] partial sums
    size_t zout_stride;
    __nv_bfloat16 *y;         // stage A output [T][rows]
    int T;
    int kt_per_cta;           // sign tiles along the reduction per blockIdx.y slice
    int WR;                   // warps along rows (1, 2 or 4); 8 / WR warps split the reduction
};

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Shared-memory plan (dynamic):
//   vbuf[2][DEC_CT * 8 * NT * 32] uint2      V fragments, double buffered
//   xp[TT][nk * 64] uint32                   activation pairs {in[c], in[c + 16]} per (tile, word, bit < 16)
//   red[WK][TT][WR * 32] float               cross-warp partial sums (aliases vbuf after the main loop)
template <int NT, int TT, bool STAGE_A>
__global__ void __launch_bounds__(DEC_THREADS, (NT * TT <= 4) ? 2 : 1) decode_stage_kernel(const StageArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int VBUF_ELEMS = DEC_CT * 8 * NT * 32;   // uint2 per buffer
    uint2 *vbuf = reinterpret_cast<uint2 *>(smem_raw);
    uint32_t *xp = reinterpret_cast<uint32_t *>(smem_raw + 2 * VBUF_ELEMS * sizeof(uint2));

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, q = lane & 3;
    const int WR = a.WR, WK = DEC_WARPS / WR;
    const int wr = warp % WR, wk = warp / WR;
    const int rt = blockIdx.x * WR + wr;
    const bool row_ok = rt < a.rtiles;
    const int kt0 = blockIdx.y * a.kt_per_cta;
    const int kt1 = min(a.ktiles, kt0 + a.kt_per_cta);
    const int nk = kt1 - kt0;                       // > 0 by construction of the grid
    const int nchunks = (nk + DEC_CT - 1) / DEC_CT;

    // ---- weights first: V chunks 0 and 1 through cp.async, sign tiles of chunk 0 into registers
    auto issue_v = [&](int chunk) {
        const int t0 = kt0 + chunk * DEC_CT;
        const int nt_tiles = min(DEC_CT, kt1 - t0);
        const int n16 = nt_tiles * 8 * NT * 32 / 2;                 // 16-byte pieces
        const uint4 *src = reinterpret_cast<const uint4 *>(a.vfrag + (size_t)t0 * 8 * NT * 32);
        uint4 *dst = reinterpret_cast<uint4 *>(vbuf + (chunk & 1) * VBUF_ELEMS);
        for (int i = tid; i < n16; i += DEC_THREADS) cp_async16(dst + i, src + i);
    };
    auto load_signs = [&](int chunk, uint4 (&s)[DEC_MAX_TPW]) {
#pragma unroll
        for (int i = 0; i < DEC_MAX_TPW; ++i) {
            const int kt = kt0 + chunk * DEC_CT + wk + i * WK;
            if (i < WR && row_ok && kt < kt1 && chunk < nchunks)
                s[i] = __ldg(a.tiled + ((size_t)rt * a.ktiles + kt) * 32 + lane);
            else
                s[i] = make_uint4(0u, 0u, 0u, 0u);
        }
    };

    issue_v(0);
    cp_async_commit();
    if (nchunks > 1) issue_v(1);
    cp_async_commit();
    uint4 cur[DEC_MAX_TPW], nxt[DEC_MAX_TPW];
    load_signs(0, cur);

    // U for this lane's rows and modes: rows rt*32 + {g, g+8, g+16, g+24}, modes nt*8 + 2q + {0,1}
    float u[4][NT][2];
#pragma unroll
    for (int rr = 0; rr < 4; ++rr) {
        const int row = rt * 32 + g + 8 * rr;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int t = nt * 8 + 2 * q + e;
                u[rr][nt][e] = (row_ok && row < a.rows && t < a.l) ? env_load(a.U, (size_t)row * a.l + t, a.env_dtype) : 0.f;
            }
    }

    pdl_launch_dependents();
    pdl_wait();            // everything below may read what earlier kernels in the stream wrote

    // ---- stage the activation pairs for this CTA's reduction range
    const int npairs = nk * 64;
    for (int idx = tid; idx < npairs * TT; idx += DEC_THREADS) {
        const int tau = idx / npairs, pi = idx - tau * npairs;
        const int ktl = pi >> 6, word = (pi >> 4) & 3, p = pi & 15;
        const int c_lo = (kt0 + ktl) * 128 + word * 32 + p, c_hi = c_lo + 16;
        float lo = 0.f, hi = 0.f;
        if (tau < a.T) {
            if (STAGE_A) {
                for (int s = 0; s < a.nsplit_in; ++s) {
                    const float *zp = a.zin + s * a.zin_stride + (size_t)tau * a.cols;
                    if (c_lo < a.cols) lo += zp[c_lo];
                    if (c_hi < a.cols) hi += zp[c_hi];
                }
            } else {
                const __nv_bfloat16 *xr = a.x + (size_t)tau * a.cols;
                if (c_lo < a.cols) lo = __bfloat162float(xr[c_lo]);
                if (c_hi < a.cols) hi = __bfloat162float(xr[c_hi]);
            }
        }
        xp[tau * npairs + pi] = pack_bf16x2(lo, hi);
    }

    float acc[TT][2][NT][4];
#pragma unroll
    for (int tau = 0; tau < TT; ++tau)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[tau][h][nt][e] = 0.f;

    // ---- main loop over chunks of DEC_CT sign tiles
    for (int chunk = 0; chunk < nchunks; ++chunk) {
        if (chunk + 1 < nchunks) cp_async_wait<1>(); else cp_async_wait<0>();
        __syncthreads();
        load_signs(chunk + 1, nxt);
        const uint2 *vb = vbuf + (chunk & 1) * VBUF_ELEMS;
#pragma unroll
        for (int i = 0; i < DEC_MAX_TPW; ++i) {
            const int ktl_c = wk + i * WK;                  // tile inside the chunk
            const int ktl = chunk * DEC_CT + ktl_c;         // tile inside the CTA's range
            if (i < WR && row_ok && ktl < nk) {
                const uint4 w = cur[i];
#pragma unroll
                for (int m = 0; m < 8; ++m) {
                    // bits (2m, 2m+16) and (2m+1, 2m+17) of each word moved to the bf16 sign positions
                    const uint32_t x0 = (w.x << (15 - 2 * m)) & 0x80008000u, x1 = (w.x << (14 - 2 * m)) & 0x80008000u;
                    const uint32_t y0 = (w.y << (15 - 2 * m)) & 0x80008000u, y1 = (w.y << (14 - 2 * m)) & 0x80008000u;
                    const uint32_t z0 = (w.z << (15 - 2 * m)) & 0x80008000u, z1 = (w.z << (14 - 2 * m)) & 0x80008000u;
                    const uint32_t w0 = (w.w << (15 - 2 * m)) & 0x80008000u, w1 = (w.w << (14 - 2 * m)) & 0x80008000u;
                    uint2 b[NT];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) b[nt] = vb[((ktl_c * 8 + m) * NT + nt) * 32 + lane];
#pragma unroll
                    for (int tau = 0; tau < TT; ++tau) {
                        const uint2 xq = *reinterpret_cast<const uint2 *>(xp + tau * npairs + ktl * 64 + q * 16 + 2 * m);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            mma_bf16_16816(acc[tau][0][nt], x0 ^ xq.x, y0 ^ xq.x, x1 ^ xq.y, y1 ^ xq.y, b[nt].x, b[nt].y);
                            mma_bf16_16816(acc[tau][1][nt], z0 ^ xq.x, w0 ^ xq.x, z1 ^ xq.y, w1 ^ xq.y, b[nt].x, b[nt].y);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < DEC_MAX_TPW; ++i) cur[i] = nxt[i];
        __syncthreads();
        if (chunk + 2 < nchunks) issue_v(chunk + 2);
        cp_async_commit();
    }

    // ---- epilogue: mode contraction with U (quad shuffle), cross-warp sum, store
    float *red = reinterpret_cast<float *>(smem_raw);      // vbuf is free after the last barrier
    const int rows_cta = WR * 32;
#pragma unroll
    for (int tau = 0; tau < TT; ++tau)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int rr = h * 2 + half;               // row g + 8*rr of the 32-row tile
                float v = 0.f;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
                    v += u[rr][nt][0] * acc[tau][h][nt][half * 2 + 0] + u[rr][nt][1] * acc[tau][h][nt][half * 2 + 1];
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                if (q == 0) red[(wk * TT + tau) * rows_cta + wr * 32 + g + 8 * rr] = v;
            }
    __syncthreads();
    for (int idx = tid; idx < TT * rows_cta; idx += DEC_THREADS) {
        const int tau = idx / rows_cta, rl = idx - tau * rows_cta;
        const int row = blockIdx.x * rows_cta + rl;
        if (tau >= a.T || row >= a.rows) continue;
        float v = 0.f;
        for (int k2 = 0; k2 < WK; ++k2) v += red[(k2 * TT + tau) * rows_cta + rl];
        if (STAGE_A) a.y[(size_t)tau * a.rows + row] = __float2bfloat16_rn(v);
        else a.zout[blockIdx.y * a.zout_stride + (size_t)tau * a.rows + row] = v;
    }
}

// bf16 copy of V (cols x l) in B-fragment order: element e of the uint2 of
// (kt, m, nt, lane = 4g + q) is V[kt*128 + 32q + bit][nt*8 + g] with
// bit = 2m, 2m+16, 2m+1, 2m+17 for e = 0..3; zero outside the matrix.
__global__ void vfrag_kernel(const void *__restrict__ V, int cols, int l, int env_dtype,
                             __nv_bfloat16 *__restrict__ out, int ktiles, int NT) {
    const size_t total = (size_t)ktiles * 8 * NT * 32 * 4;
    for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (size_t)gridDim.x * blockDim.x) {
        const int e = (int)(idx & 3);
        const int lane = (int)((idx >> 2) & 31);
        size_t rest = idx >> 7;
        const int nt = (int)(rest % NT); rest /= NT;
        const int m = (int)(rest & 7);
        const int kt = (int)(rest >> 3);
        const int g = lane >> 2, q = lane & 3;
        const int bit = 2 * m + (e >> 1) + 16 * (e & 1);
        const int c = kt * 128 + 32 * q + bit;
        const int t = nt * 8 + g;
        float v = 0.f;
        if (c < cols && t < l) v = env_load(V, (size_t)c * l + t, env_dtype);
        out[idx] = __float2bfloat16_rn(v);
    }
}

mdbf_status_t launch_vfrag(const void *V, int cols, int l, int env_dtype, uint2 *out, int ktiles, int NT,
                           cudaStream_t st) {
    const size_t total = (size_t)ktiles * 8 * NT * 32 * 4;
    int grid = (int)((total + 255) / 256);
    if (grid > 148 * 16) grid = 148 * 16;
    vfrag_kernel<<<grid, 256, 0, st>>>(V, cols, l, env_dtype, reinterpret_cast<__nv_bfloat16 *>(out), ktiles, NT);
    MDBF_CUDA(cudaGetLastError());
    return MDBF_OK;
}

// ---------------------------------------------------------------------------
static bool pdl_enabled() {
    static int v = -1;
    if (v < 0) {
        const char *e = getenv("MDBF_PDL");
        v = (e && e[0] == '0') ? 0 : 1;
    }
    return v == 1;
}

template <int NT, int TT, bool STAGE_A>
static mdbf_status_t launch_stage(const StageArgs &a, dim3 grid, cudaStream_t st) {
    const int nk_max = a.kt_per_cta;
    const size_t vbytes = 2 * (size_t)DEC_CT * 8 * NT * 32 * sizeof(uint2);
    const size_t xbytes = (size_t)TT * nk_max * 64 * sizeof(uint32_t);
    const size_t smem = vbytes + xbytes;
    auto kern = decode_stage_kernel<NT, TT, STAGE_A>;
    static bool attr_set = false;          // per instantiation
    if (!attr_set) {
        MDBF_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        attr_set = true;
    }
    if (smem > 200 * 1024) {
        set_error("decode stage: reduction range of %d tiles needs %zu bytes of shared memory", nk_max, smem);
        return MDBF_ERR_SHAPE;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(DEC_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    MDBF_CUDA(cudaLaunchKernelEx(&cfg, kern, a));
    return MDBF_OK;
}

template <bool STAGE_A>
static mdbf_status_t dispatch_stage(int NT, int T, const StageArgs &a, dim3 grid, cudaStream_t st) {
    const int TT = T <= 1 ? 1 : T <= 2 ? 2 : 4;
#define MDBF_CASE(nt, tt) \
    if (NT == nt && TT == tt) return launch_stage<nt, tt, STAGE_A>(a, grid, st);
    MDBF_CASE(1, 1) MDBF_CASE(1, 2) MDBF_CASE(1, 4)
    MDBF_CASE(2, 1) MDBF_CASE(2, 2) MDBF_CASE(2, 4)
    MDBF_CASE(4, 1) MDBF_CASE(4, 2) MDBF_CASE(4, 4)
#undef MDBF_CASE
    set_error("decode stage: unsupported mode-tile count %d", NT);
    return MDBF_ERR_SHAPE;
}

// Grid shape: WR warps along rows (more rows per CTA = fewer re-reads of V from
// L2), the reduction split over blockIdx.y for stage B only (stage A writes y
// directly).  Aim for at least ~2 CTAs per SM, keep reduction slices whole chunks.
static void plan(int rtiles, int ktiles, bool allow_ksplit, int *WR, int *ksplit, int *kt_per_cta) {
    const int target = 148 * 2;
    int best_wr = 1, best_ks = 1;
    for (int wr = 4; wr >= 1; wr >>= 1) {
        const int rows_ctas = ceil_div(rtiles, wr);
        int ks = 1;
        if (allow_ksplit) {
            const int max_ks = min(kMaxKSplit, ceil_div(ktiles, DEC_CT));
            ks = min(max_ks, max(1, ceil_div(target, rows_ctas)));
        }
        best_wr = wr; best_ks = ks;
        if (rows_ctas * ks >= target || wr == 1) break;
    }
    int per = ceil_div(ktiles, best_ks);
    per = ceil_div(per, DEC_CT) * DEC_CT;          // whole chunks per slice
    best_ks = ceil_div(ktiles, per);
    *WR = best_wr; *ksplit = best_ks; *kt_per_cta = per;
}

mdbf_status_t launch_forward_decode(Layer &L, const void *x, void *y, int T, cudaStream_t st, int *launches) {
    const mdbf_desc_t &d = L.d;
    // stage B: rows = k, cols = d_in
    StageArgs b = {};
    int ksplit = 1;
    plan(L.rtB, L.ktB, true, &b.WR, &ksplit, &b.kt_per_cta);
    b.tiled = reinterpret_cast<const uint4 *>(L.tB); b.rtiles = L.rtB; b.ktiles = L.ktB;
    b.vfrag = L.vfB; b.U = L.UB; b.env_dtype = d.env_dtype; b.l = d.l;
    b.rows = d.k; b.cols = d.d_in;
    b.x = reinterpret_cast<const __nv_bfloat16 *>(x);
    b.zout = L.z; b.zout_stride = L.zstride; b.T = T;
    mdbf_status_t rc = dispatch_stage<false>(L.NT, T, b, dim3(ceil_div(L.rtB, b.WR), ksplit), st);
    if (rc) return rc;
    // stage A: rows = d_out, cols = k
    StageArgs a = {};
    int one = 1;
    plan(L.rtA, L.ktA, false, &a.WR, &one, &a.kt_per_cta);
    a.tiled = reinterpret_cast<const uint4 *>(L.tA); a.rtiles = L.rtA; a.ktiles = L.ktA;
    a.vfrag = L.vfA; a.U = L.UA; a.env_dtype = d.env_dtype; a.l = d.l;
    a.rows = d.d_out; a.cols = d.k;
    a.zin = L.z; a.nsplit_in = ksplit; a.zin_stride = L.zstride;
    a.y = reinterpret_cast<__nv_bfloat16 *>(y); a.T = T;
    rc = dispatch_stage<true>(L.NT, T, a, dim3(ceil_div(L.rtA, a.WR), 1), st);
    if (rc) return rc;
    L.last_ksplit = ksplit;
    *launches = 2;
    return MDBF_OK;
}

}  // namespace mdbf
