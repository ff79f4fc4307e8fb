// C-ABI entry points of libmdbf: argument checking, handle lifetime, dispatch.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"

namespace mdbf {

static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

mdbf_status_t cuda_fail(cudaError_t e, const char *what) {
    set_error("CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
    if (e == cudaErrorMemoryAllocation) return MDBF_ERR_ALLOC;
    return MDBF_ERR_CUDA;
}

// The product has no CPU fallback: anything that computes needs an sm_100 device.
mdbf_status_t require_device(int *dev_out) {
    int n = 0;
    cudaError_t e = cudaGetDeviceCount(&n);
    if (e != cudaSuccess || n == 0) {
        cudaGetLastError();
        set_error("libmdbf needs a CUDA device of compute capability 10.x; none is visible (%s)",
                  e == cudaSuccess ? "device count 0" : cudaGetErrorString(e));
        return MDBF_ERR_ARCH;
    }
    int dev = 0;
    MDBF_CUDA(cudaGetDevice(&dev));
    int major = 0;
    MDBF_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    if (major != 10) {
        set_error("libmdbf is built for sm_100a only; device %d has compute capability major %d", dev, major);
        return MDBF_ERR_ARCH;
    }
    if (dev_out) *dev_out = dev;
    return MDBF_OK;
}

static bool valid_dtype(int dt) { return dt == MDBF_F32 || dt == MDBF_F16 || dt == MDBF_BF16; }

static mdbf_status_t check_handle(mdbf_handle_t h, const char *fn) {
    if (h == nullptr || h->magic != kHandleMagic) {
        set_error("%s: invalid handle", fn);
        return MDBF_ERR_INVALID_ARG;
    }
    return MDBF_OK;
}

// A layer lives on the device it was packed on; its kernels must be launched there.
static mdbf_status_t check_device(const Layer &L, const char *fn) {
    int dev = -1;
    MDBF_CUDA(cudaGetDevice(&dev));
    if (dev != L.device) {
        set_error("%s: the layer was packed on device %d, the current device is %d", fn, L.device, dev);
        return MDBF_ERR_INVALID_ARG;
    }
    return MDBF_OK;
}

}  // namespace mdbf
mdbf::SignView mdbf::sign_view(const Layer &L, int which) {
    SignView v;
    v.canon = which == 0 ? L.wA : L.wB;
    v.wk2 = which == 0 ? L.wk2A : L.wk2B;
    v.nwords = which == 0 ? L.wordsA : L.wordsB;
    v.kb_pad = which == 0 ? L.kbpA : L.kbpB;
    return v;
}
namespace mdbf {

static void free_layer(Layer &L) {
    void *ptrs[] = {L.wA, L.wB, L.UA, L.VA, L.UB, L.VB, L.vxA, L.vxB, L.wk2A, L.wk2B, L.wkA, L.wkB, L.uiA, L.uiB, L.viA, L.viB, L.vtB, L.xsB, L.xsA, L.zb, L.zsum, L.xstage, L.ystage, L.status};
    for (void *p : ptrs)
        if (p) cudaFree(p);
    t1_release(L);
}

// mdbf_pack builds what the default dispatch uses (canonical words, the row-block-major sign copy, the
// one-token V tiles, the envelope images).  The private layouts and scratch of the other kernels are built
// here on their first use (or by mdbf_set_kernel): on the default stream, followed by a synchronisation.
#define ENS_CUDA(call)                                                   \
    do {                                                                 \
        cudaError_t e__ = (call);                                        \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call);            \
    } while (0)
#define ENS_RC(call)                                 \
    do {                                             \
        mdbf_status_t r__ = (call);                  \
        if (r__ != MDBF_OK) return r__;              \
    } while (0)
static mdbf_status_t ensure_kblock_words(Layer &L) {
    const mdbf_desc_t &d = L.d;
    if (L.wkA) return MDBF_OK;
    uint2 *a = nullptr, *b = nullptr;
    ENS_CUDA(dev_malloc(&a, (size_t)(L.padA / 64) * L.rpA * sizeof(uint2)));
    cudaError_t e = dev_malloc(&b, (size_t)(L.padB / 64) * L.rpB * sizeof(uint2));
    if (e != cudaSuccess) { cudaFree(a); return cuda_fail(e, "K-blocked sign words"); }
    mdbf_status_t rc = launch_kblock(sign_view(L, 0), d.d_out, a, L.rpA, L.padA / 64, 0);
    if (rc == MDBF_OK) rc = launch_kblock(sign_view(L, 1), d.k, b, L.rpB, L.padB / 64, 0);
    if (rc) { cudaFree(a); cudaFree(b); return rc; }
    L.wkA = a; L.wkB = b;
    return MDBF_OK;
}
// Scratch and private layouts of the expanded-order kernel (K-blocked sign words, transposed V_B, the pre-scaled
// operands): built by mdbf_pack for layers that can only run that order, else by mdbf_set_kernel(PREFILL) - never
// by a forward.  Every buffer is published to the layer only once it is complete.
mdbf_status_t ensure_kernel_layouts(Layer &L, int kernel, int T) {
    (void)T;
    const mdbf_desc_t &d = L.d;
    if (kernel != MDBF_KERNEL_PREFILL || !L.zb || L.xsB) return MDBF_OK;
    ENS_RC(ensure_kblock_words(L));
    if (!L.vtB) {
        float *vt = nullptr;
        ENS_CUDA(dev_malloc(&vt, (size_t)L.LP * L.padB * sizeof(float)));
        mdbf_status_t rc = launch_vtrans(L.VB, d.d_in, d.l, d.env_dtype, vt, L.padB, L.LP, 0);
        if (rc) { cudaFree(vt); return rc; }
        L.vtB = vt;
    }
    ENS_RC(ensure_prefill_scratch(L));
    ENS_CUDA(cudaStreamSynchronize(0));
    return MDBF_OK;
}
static mdbf_status_t ensure_host_staging(Layer &L) {
    if (L.xstage) return MDBF_OK;
    void *xs = nullptr, *ys = nullptr;
    ENS_CUDA(dev_malloc(&xs, (size_t)L.d.max_T * L.d.d_in * 4));
    cudaError_t e = dev_malloc(&ys, (size_t)L.d.max_T * L.d.d_out * 4);
    if (e != cudaSuccess) { cudaFree(xs); return cuda_fail(e, "host-entry staging"); }
    L.xstage = xs; L.ystage = ys;
    return MDBF_OK;
}
#undef ENS_CUDA
#undef ENS_RC

static thread_local int g_fail_alloc_in = 0;       // > 0: that many dev_malloc calls from now, the last of them fails
cudaError_t dev_malloc(void **p, size_t bytes) {
    if (g_fail_alloc_in > 0 && --g_fail_alloc_in == 0) {
        *p = nullptr;
        return cudaErrorMemoryAllocation;
    }
    return cudaMalloc(p, bytes);
}

}  // namespace mdbf

using namespace mdbf;

extern "C" {

void mdbf_debug_fail_alloc(int nth) { g_fail_alloc_in = nth > 0 ? nth : 0; }

const char *mdbf_last_error(void) { return g_err; }
const char *mdbf_version(void) {
#ifdef MDBF_BOUNDS_CHECK
    return "libmdbf 0.2 (sm_100a) +bounds-check";
#else
    return "libmdbf 0.2 (sm_100a)";
#endif
}

mdbf_status_t mdbf_pack_signs(const int8_t *s, int64_t rows, int64_t cols, uint32_t *out, int on_device,
                              void *stream) {
    if (!s || !out) { set_error("mdbf_pack_signs: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    if (rows < 0 || cols < 0) { set_error("mdbf_pack_signs: negative size"); return MDBF_ERR_SHAPE; }
    if (rows == 0 || cols == 0) return MDBF_OK;
    if (!on_device) return host_pack(s, rows, cols, out);
    mdbf_status_t rc = require_device(nullptr);
    if (rc) return rc;
    return launch_pack(s, rows, cols, out, (cudaStream_t)stream);
}

mdbf_status_t mdbf_unpack_signs(const uint32_t *p, int64_t rows, int64_t cols, int8_t *out, int on_device,
                                void *stream) {
    if (!p || !out) { set_error("mdbf_unpack_signs: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    if (rows < 0 || cols < 0) { set_error("mdbf_unpack_signs: negative size"); return MDBF_ERR_SHAPE; }
    if (rows == 0 || cols == 0) return MDBF_OK;
    if (!on_device) return host_unpack(p, rows, cols, out);
    mdbf_status_t rc = require_device(nullptr);
    if (rc) return rc;
    return launch_unpack(p, rows, cols, out, (cudaStream_t)stream);
}

mdbf_status_t mdbf_pack(const mdbf_desc_t *desc, const int8_t *S_A, const int8_t *S_B, const float *U_A,
                        const float *V_A, const float *U_B, const float *V_B, int inputs_on_device,
                        void *stream, mdbf_handle_t *out) {
    if (!desc || !S_A || !S_B || !U_A || !V_A || !U_B || !V_B || !out) {
        set_error("mdbf_pack: NULL pointer");
        return MDBF_ERR_INVALID_ARG;
    }
    *out = nullptr;
    const mdbf_desc_t d = *desc;
    if (d.d_out < 1 || d.d_in < 1 || d.k < 1 || d.l < 1 || d.l > kMaxL || d.max_T < 1) {
        set_error("mdbf_pack: bad shape d_out=%d d_in=%d k=%d l=%d max_T=%d (need all >= 1, l <= %d)",
                  d.d_out, d.d_in, d.k, d.l, d.max_T, kMaxL);
        return MDBF_ERR_SHAPE;
    }
    if (!valid_dtype(d.env_dtype)) { set_error("mdbf_pack: bad env_dtype %d", d.env_dtype); return MDBF_ERR_DTYPE; }
    int dev = 0;
    mdbf_status_t rc = require_device(&dev);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;

    if (!inputs_on_device) {   // validate host signs before touching the device
        const int8_t *mats[2] = {S_A, S_B};
        const size_t cnt[2] = {(size_t)d.d_out * d.k, (size_t)d.k * d.d_in};
        for (int m = 0; m < 2; ++m)
            for (size_t e = 0; e < cnt[m]; ++e)
                if (mats[m][e] != 1 && mats[m][e] != -1) {
                    set_error("mdbf_pack: S_%c entry %zu is %d, expected +1 or -1", m ? 'B' : 'A', e, (int)mats[m][e]);
                    return MDBF_ERR_VALUE;
                }
    }

    mdbf_handle_s *h = new (std::nothrow) mdbf_handle_s();
    if (!h) { set_error("mdbf_pack: host allocation failed"); return MDBF_ERR_ALLOC; }
    memset(h, 0, sizeof(*h));
    Layer &L = h->L;
    L.d = d;
    L.device = dev;
    L.wordsA = ceil_div(d.k, 32);
    L.wordsB = ceil_div(d.d_in, 32);
    const size_t es = dtype_size(d.env_dtype);
    const size_t nUA = (size_t)d.d_out * d.l, nVA = (size_t)d.k * d.l, nUB = nVA, nVB = (size_t)d.d_in * d.l;
    const size_t nSA = (size_t)d.d_out * d.k, nSB = (size_t)d.k * d.d_in;

    std::vector<void *> temps;
    auto fail = [&](mdbf_status_t code) {
        for (void *p : temps) cudaFree(p);
        free_layer(L);
        delete h;
        return code;
    };
#define PACK_CUDA(call)                                                  \
    do {                                                                 \
        cudaError_t e__ = (call);                                        \
        if (e__ != cudaSuccess) return fail(cuda_fail(e__, #call));      \
    } while (0)
#define PACK_RC(call)                                \
    do {                                             \
        mdbf_status_t r__ = (call);                  \
        if (r__ != MDBF_OK) return fail(r__);        \
    } while (0)

    PACK_CUDA(dev_malloc(&L.wA, (size_t)d.d_out * L.wordsA * 4));
    PACK_CUDA(dev_malloc(&L.wB, (size_t)d.k * L.wordsB * 4));
    PACK_CUDA(dev_malloc(&L.UA, nUA * es));
    PACK_CUDA(dev_malloc(&L.VA, nVA * es));
    PACK_CUDA(dev_malloc(&L.UB, nUB * es));
    PACK_CUDA(dev_malloc(&L.VB, nVB * es));
    L.LP = 1;
    while (L.LP < d.l) L.LP *= 2;
    L.padA = ceil_div(d.k, 64) * 64; L.padB = ceil_div(d.d_in, 64) * 64;
    L.rpA = ceil_div(d.d_out, 128) * 128; L.rpB = ceil_div(d.k, 128) * 128;
    // the large-T kernel takes 16-bit envelopes and l <= 32; its scratch is sized by max_T
    const bool want_prefill = d.env_dtype != MDBF_F32 && d.l <= 32 && d.max_T >= 2;
    const bool want_tc = d.env_dtype != MDBF_F32 && d.l <= 32;
    if (want_tc) {
        const int NB = L.LP < 16 ? 16 : L.LP;
        L.kbpA = ceil_div(L.padA / 64, 2) * 2; L.kbpB = ceil_div(L.padB / 64, 2) * 2;
        PACK_CUDA(dev_malloc(&L.vxA, (size_t)L.kbpA * NB * 64 * sizeof(uint16_t)));
        PACK_CUDA(dev_malloc(&L.vxB, (size_t)L.kbpB * NB * 64 * sizeof(uint16_t)));
        PACK_CUDA(dev_malloc(&L.wk2A, (size_t)(L.rpA / 128) * L.kbpA * 128 * sizeof(uint2)));
        PACK_CUDA(dev_malloc(&L.wk2B, (size_t)(L.rpB / 128) * L.kbpB * 128 * sizeof(uint2)));
    }
    if (want_prefill) {
        // The pre-scaled operands of the expanded order (max_T * LP * (d_in + k) * 2 bytes) are allocated on
        // its first use (ensure_prefill_scratch): the default path for T >= 2 does not need them.
        // bf16 intermediate of the materialised-envelope kernels, [max_T][padA]; the padding columns stay zero
        PACK_CUDA(dev_malloc(&L.zb, (size_t)d.max_T * L.padA * 2));
        PACK_CUDA(cudaMemsetAsync(L.zb, 0, (size_t)d.max_T * L.padA * 2, st));
        L.kcm = d.l <= 16 ? 2 : 4;
        PACK_CUDA(dev_malloc(&L.uiA, (size_t)(L.rpA / 128) * L.kcm * 1024 * sizeof(uint16_t)));
        PACK_CUDA(dev_malloc(&L.uiB, (size_t)(L.rpB / 128) * L.kcm * 1024 * sizeof(uint16_t)));
        PACK_CUDA(dev_malloc(&L.viA, (size_t)ceil_div(L.padA, 128) * L.kcm * 1024 * sizeof(uint16_t)));
        PACK_CUDA(dev_malloc(&L.viB, (size_t)ceil_div(L.padB, 128) * L.kcm * 1024 * sizeof(uint16_t)));
    }
    PACK_CUDA(dev_malloc(&L.zsum, (size_t)d.max_T * d.k * sizeof(float)));
    PACK_CUDA(dev_malloc(&L.status, sizeof(int32_t)));
    PACK_CUDA(cudaMemsetAsync(L.status, 0, sizeof(int32_t), st));
    PACK_CUDA(cudaMemsetAsync(L.zsum, 0, (size_t)d.max_T * d.k * sizeof(float), st));

    // bring inputs to the device if needed
    const void *src[6] = {S_A, S_B, U_A, V_A, U_B, V_B};
    const size_t bytes[6] = {nSA, nSB, nUA * 4, nVA * 4, nUB * 4, nVB * 4};
    const void *dsrc[6];
    for (int i = 0; i < 6; ++i) {
        if (inputs_on_device) { dsrc[i] = src[i]; continue; }
        void *tmp = nullptr;
        PACK_CUDA(dev_malloc(&tmp, bytes[i]));
        temps.push_back(tmp);
        PACK_CUDA(cudaMemcpyAsync(tmp, src[i], bytes[i], cudaMemcpyHostToDevice, st));
        dsrc[i] = tmp;
    }
    PACK_RC(launch_pack((const int8_t *)dsrc[0], d.d_out, d.k, L.wA, st));
    PACK_RC(launch_pack((const int8_t *)dsrc[1], d.k, d.d_in, L.wB, st));
    PACK_RC(launch_env_round((const float *)dsrc[2], L.UA, nUA, d.env_dtype, st));
    PACK_RC(launch_env_round((const float *)dsrc[3], L.VA, nVA, d.env_dtype, st));
    PACK_RC(launch_env_round((const float *)dsrc[4], L.UB, nUB, d.env_dtype, st));
    PACK_RC(launch_env_round((const float *)dsrc[5], L.VB, nVB, d.env_dtype, st));
    if (want_tc) {
        PACK_RC(launch_vtile(L.VA, d.k, d.l, d.env_dtype, L.vxA, L.kbpA, L.LP < 16 ? 16 : L.LP, st));
        PACK_RC(launch_vtile(L.VB, d.d_in, d.l, d.env_dtype, L.vxB, L.kbpB, L.LP < 16 ? 16 : L.LP, st));
        PACK_RC(launch_wk2(L.wA, d.d_out, L.wordsA, L.wk2A, L.rpA / 128, L.kbpA, st));
        PACK_RC(launch_wk2(L.wB, d.k, L.wordsB, L.wk2B, L.rpB / 128, L.kbpB, st));
        if (L.LP <= 16) PACK_RC(t1_prepare(L, st));
    }
    if (want_prefill) {
        PACK_RC(launch_uimg(L.UA, d.d_out, d.l, d.env_dtype, L.uiA, L.rpA / 128, L.kcm, st));
        PACK_RC(launch_uimg(L.UB, d.k, d.l, d.env_dtype, L.uiB, L.rpB / 128, L.kcm, st));
        PACK_RC(launch_uimg(L.VA, d.k, d.l, d.env_dtype, L.viA, ceil_div(L.padA, 128), L.kcm, st));     // V: columns of a pair of K blocks as rows
        PACK_RC(launch_uimg(L.VB, d.d_in, d.l, d.env_dtype, L.viB, ceil_div(L.padB, 128), L.kcm, st));
    }
    PACK_CUDA(cudaStreamSynchronize(st));
    for (void *p : temps) cudaFree(p);
    temps.clear();
    if (want_tc) {                                    // one copy of the signs per layer: the row-block-major one serves every kernel
        cudaFree(L.wA); cudaFree(L.wB);
        L.wA = nullptr; L.wB = nullptr;
    }
    // a layer the materialised order can never serve (no tensor map over x) will run the expanded order
    if (want_prefill && d.d_in % 8 != 0) PACK_RC(ensure_kernel_layouts(L, MDBF_KERNEL_PREFILL, 2));
#undef PACK_CUDA
#undef PACK_RC
    h->magic = kHandleMagic;
    h->kernel = MDBF_KERNEL_AUTO;
    *out = h;
    return MDBF_OK;
}

mdbf_status_t mdbf_get_packed(mdbf_handle_t h, int which, uint32_t *out, int out_on_device, void *stream) {
    mdbf_status_t rc = check_handle(h, "mdbf_get_packed");
    if (rc) return rc;
    if (!out || (which != 0 && which != 1)) { set_error("mdbf_get_packed: bad argument"); return MDBF_ERR_INVALID_ARG; }
    const Layer &L = h->L;
    const int rows = which == 0 ? L.d.d_out : L.d.k;
    const size_t bytes = (size_t)rows * (which == 0 ? L.wordsA : L.wordsB) * 4;
    cudaStream_t st = (cudaStream_t)stream;
    const SignView sv = sign_view(L, which);
    if (out_on_device) {
        rc = launch_canon(sv, rows, out, st);
        if (rc) return rc;
        MDBF_CUDA(cudaStreamSynchronize(st));
        return MDBF_OK;
    }
    uint32_t *tmp = nullptr;                          // check path: a temporary device copy in canonical order
    MDBF_CUDA(dev_malloc(&tmp, bytes));
    rc = launch_canon(sv, rows, tmp, st);
    cudaError_t e = cudaSuccess;
    if (rc == MDBF_OK) e = cudaMemcpyAsync(out, tmp, bytes, cudaMemcpyDeviceToHost, st);
    if (rc == MDBF_OK && e == cudaSuccess) e = cudaStreamSynchronize(st);
    cudaFree(tmp);
    if (rc) return rc;
    if (e != cudaSuccess) return cuda_fail(e, "mdbf_get_packed copy");
    return MDBF_OK;
}

mdbf_status_t mdbf_get_envelope(mdbf_handle_t h, int which, float *out, int out_on_device, void *stream) {
    mdbf_status_t rc = check_handle(h, "mdbf_get_envelope");
    if (rc) return rc;
    if (!out || which < 0 || which > 3) { set_error("mdbf_get_envelope: bad argument"); return MDBF_ERR_INVALID_ARG; }
    const Layer &L = h->L;
    const void *src[4] = {L.UA, L.VA, L.UB, L.VB};
    const size_t n[4] = {(size_t)L.d.d_out * L.d.l, (size_t)L.d.k * L.d.l, (size_t)L.d.k * L.d.l,
                         (size_t)L.d.d_in * L.d.l};
    cudaStream_t st = (cudaStream_t)stream;
    if (out_on_device) {
        rc = launch_env_read(src[which], out, n[which], L.d.env_dtype, st);
        if (rc) return rc;
        MDBF_CUDA(cudaStreamSynchronize(st));
        return MDBF_OK;
    }
    float *tmp = nullptr;
    MDBF_CUDA(dev_malloc(&tmp, n[which] * 4));
    rc = launch_env_read(src[which], tmp, n[which], L.d.env_dtype, st);
    cudaError_t e = cudaSuccess;
    if (rc == MDBF_OK) e = cudaMemcpyAsync(out, tmp, n[which] * 4, cudaMemcpyDeviceToHost, st);
    if (rc == MDBF_OK && e == cudaSuccess) e = cudaStreamSynchronize(st);
    cudaFree(tmp);
    if (rc) return rc;
    if (e != cudaSuccess) return cuda_fail(e, "mdbf_get_envelope copy");
    return MDBF_OK;
}

mdbf_status_t mdbf_get_desc(mdbf_handle_t h, mdbf_desc_t *out) {
    mdbf_status_t rc = check_handle(h, "mdbf_get_desc");
    if (rc) return rc;
    if (!out) { set_error("mdbf_get_desc: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    *out = h->L.d;
    return MDBF_OK;
}

mdbf_status_t mdbf_set_kernel(mdbf_handle_t h, int32_t kernel) {
    mdbf_status_t rc = check_handle(h, "mdbf_set_kernel");
    if (rc) return rc;
    if (kernel < MDBF_KERNEL_AUTO || kernel > MDBF_KERNEL_I8 || kernel == 2) {
        set_error("mdbf_set_kernel: unknown kernel %d", kernel);
        return MDBF_ERR_INVALID_ARG;
    }
    // the expanded-order kernel's layouts and scratch are built here, never inside a forward
    if (kernel == MDBF_KERNEL_PREFILL && h->L.wk2A != nullptr) {
        rc = ensure_kernel_layouts(h->L, kernel, 2);
        if (rc) return rc;
    }
    h->kernel = kernel;
    return MDBF_OK;
}

// One token, n <= 4 layers that share x and are prepared for both one-token kernels.  Each stage goes to the kernel
// that is faster for its size: the integer kernel streams a stage's sign words several times faster but needs two
// launches per stage (operand images, then the contraction); below kI8StageBytes of sign words per stage the
// single launch of the bf16 TMEM-operand kernel wins.  The two kernels exchange the intermediate through the
// layers' fp32 z buffers, so the stages can mix.  force: 0 = choose, 1 = TMEM-operand kernel, 2 = integer kernel.
static constexpr size_t kI8StageBytes = 18u << 20;
static mdbf_status_t forward_t1_auto(Layer *const *Ls, int n, const void *x, void *const *ys, cudaStream_t st, int force,
                                     int *launches, int *kernel_used) {
    size_t bytes[2] = {0, 0};
    bool i8_ok = true, old_ok = true;
    for (int i = 0; i < n; ++i) {
        bytes[0] += (size_t)Ls[i]->d.k * Ls[i]->d.d_in / 8;
        bytes[1] += (size_t)Ls[i]->d.d_out * Ls[i]->d.k / 8;
        i8_ok = i8_ok && t1_supports(*Ls[i]) && Ls[i]->out_mode == 0;
        old_ok = old_ok && Ls[i]->vxA && Ls[i]->vxB && tmem_path_supports(*Ls[i], 1);
    }
    int i8_stages = 0;
    for (int s = 0; s < 2; ++s)
        if (i8_ok && (force == 2 || !old_ok || (force == 0 && bytes[s] >= kI8StageBytes))) i8_stages |= 1 << s;
    if (!i8_ok && !old_ok) { set_error("mdbf_linear_forward: no one-token kernel fits this layer"); return MDBF_ERR_SHAPE; }
    const void *xs[kMaxSiblings];
    for (int i = 0; i < n; ++i) xs[i] = x;
    int nl = 0;
    for (int s = 0; s < 2; ++s) {
        mdbf_status_t rc;
        if (i8_stages >> s & 1) { rc = launch_forward_t1_group(Ls, n, xs, ys, st, 1 << s); nl += 2; }
        else { rc = launch_forward_tmem_t1_multi(Ls, n, x, ys, st, 1 << s); nl += last_t1_launch_count(); }
        if (rc) return rc;
    }
    *launches = nl;
    *kernel_used = i8_stages == 3 ? MDBF_KERNEL_I8 : MDBF_KERNEL_TMEM;
    return MDBF_OK;
}

static mdbf_status_t forward_impl(mdbf_handle_t h, const void *x, void *y, int32_t T, int32_t act_dtype,
                                  cudaStream_t st, int out_mode = 0) {
    Layer &L = h->L;
    L.out_mode = out_mode;
    if (T < 1 || T > L.d.max_T) {
        set_error("mdbf_linear_forward: T=%d outside [1, max_T=%d]", T, L.d.max_T);
        return MDBF_ERR_SHAPE;
    }
    if (!valid_dtype(act_dtype)) { set_error("mdbf_linear_forward: bad act_dtype %d", act_dtype); return MDBF_ERR_DTYPE; }
    {
        mdbf_status_t rcd = check_device(L, "mdbf_linear_forward");
        if (rcd) return rcd;
    }
    int kernel = h->kernel;
    const bool tc_ok = (act_dtype == MDBF_BF16) && (L.d.env_dtype != MDBF_F32) && L.d.l <= 32;
    if (kernel == MDBF_KERNEL_AUTO) {
        // one token: TMEM-operand kernel; more: the tcgen05 GEMM (it splits the reduction over a
        // cluster when few tokens would leave SMs idle); the others remain selectable
        if (!tc_ok) kernel = MDBF_KERNEL_ALU;
        else if (T == 1 && out_mode == 0 && (t1_supports(L) || tmem_path_supports(L, T))) kernel = -1;     // one token: per-stage choice below
        else if (T == 1 && tmem_path_supports(L, T)) kernel = MDBF_KERNEL_TMEM;
        // more tokens: rebuilding W_hat tiles and running one GEMM of width T (measured faster than, or equal
        // to, the l sign GEMMs of the expanded order at every T >= 2); the expanded order serves the layers
        // the tensor map over x cannot take (d_in not a multiple of 8, unaligned x)
        else if (mat_path_supports(L, x, T)) kernel = MDBF_KERNEL_MAT;
        else if (L.xsB) kernel = MDBF_KERNEL_PREFILL;           // its scratch exists (d_in % 8 != 0 layers get it at pack time)
        else kernel = MDBF_KERNEL_ALU;                          // e.g. an x that is not 16-byte aligned: no allocation here, ever
    }
    if (kernel == -1) {
        Layer *one = &L;
        int launches = 0, used = 0;
        mdbf_status_t rc = forward_t1_auto(&one, 1, x, &y, st, 0, &launches, &used);
        if (rc == MDBF_OK) { L.last_ksplit = 0; h->last_launches = launches; h->last_kernel = used; }
        return rc;
    }
    if (kernel != MDBF_KERNEL_ALU && !tc_ok) {
        set_error("mdbf_linear_forward: the tensor-core kernels need bf16 activations, 16-bit envelopes and l <= 32");
        return MDBF_ERR_DTYPE;
    }
    if (kernel == MDBF_KERNEL_PREFILL && !L.xsB) {
        set_error("mdbf_linear_forward: the expanded-order kernel has no scratch on this handle; call mdbf_set_kernel(handle, MDBF_KERNEL_PREFILL) first (it allocates; a handle packed with max_T = 1 never has any)");
        return MDBF_ERR_INVALID_ARG;
    }
    if (kernel == MDBF_KERNEL_I8 && (T != 1 || !t1_supports(L))) {
        set_error("mdbf_linear_forward: the one-token integer kernel needs T = 1, 16-bit envelopes and l <= 32");
        return MDBF_ERR_SHAPE;
    }
    if (out_mode != 0 && kernel == MDBF_KERNEL_I8) {
        set_error("mdbf_linear_forward_sum: the forced kernel has no fp32-accumulate output");
        return MDBF_ERR_INVALID_ARG;
    }
    int launches = 0;
    mdbf_status_t rc = MDBF_OK;
    if (kernel == MDBF_KERNEL_I8) {
        Layer *one = &L;
        rc = launch_forward_t1_group(&one, 1, &x, &y, st);
        L.last_ksplit = 0;
        launches = 4;                                         // image and stage kernel, twice
    } else if (kernel == MDBF_KERNEL_ALU) rc = launch_forward_alu(L, x, y, T, act_dtype, st, &launches);
    else if (kernel == MDBF_KERNEL_TMEM) rc = launch_forward_tmem(L, x, y, T, st, &launches);
    else if (kernel == MDBF_KERNEL_MAT) rc = launch_forward_mat(L, x, y, T, st, &launches);
    else rc = launch_forward_prefill(L, x, y, T, st, &launches);
    if (rc == MDBF_OK) { h->last_launches = launches; h->last_kernel = kernel; }
    return rc;
}

mdbf_status_t mdbf_linear_forward(mdbf_handle_t h, const void *x, void *y, int32_t T, int32_t act_dtype,
                                  void *stream) {
    mdbf_status_t rc = check_handle(h, "mdbf_linear_forward");
    if (rc) return rc;
    if (!x || !y) { set_error("mdbf_linear_forward: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    return forward_impl(h, x, y, T, act_dtype, (cudaStream_t)stream);
}

mdbf_status_t mdbf_linear_forward_sum(const mdbf_handle_t *terms, int32_t P, const void *x, void *y, float *acc,
                                      int32_t T, int32_t act_dtype, void *stream) {
    if (!terms || !x || !y || !acc) { set_error("mdbf_linear_forward_sum: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    if (P < 1 || P > 64) { set_error("mdbf_linear_forward_sum: P=%d outside [1, 64]", P); return MDBF_ERR_SHAPE; }
    for (int p = 0; p < P; ++p) {
        mdbf_status_t rc = check_handle(terms[p], "mdbf_linear_forward_sum");
        if (rc) return rc;
        rc = check_device(terms[p]->L, "mdbf_linear_forward_sum");
        if (rc) return rc;
        if (terms[p]->L.d.d_out != terms[0]->L.d.d_out || terms[p]->L.d.d_in != terms[0]->L.d.d_in) {
            set_error("mdbf_linear_forward_sum: term %d is %d x %d, term 0 is %d x %d", p, terms[p]->L.d.d_out,
                      terms[p]->L.d.d_in, terms[0]->L.d.d_out, terms[0]->L.d.d_in);
            return MDBF_ERR_SHAPE;
        }
        for (int q = 0; q < p; ++q)
            if (terms[q] == terms[p]) { set_error("mdbf_linear_forward_sum: term %d repeats term %d", p, q); return MDBF_ERR_INVALID_ARG; }
    }
    cudaStream_t st = (cudaStream_t)stream;
    // One token, bf16, every term ready for the one-token kernel with the same envelope-rank bucket: stage B of
    // all terms shares a launch, the last term's stage-A epilogue adds the fp32 sum of the others and rounds
    // into y (P + 1 launches, no cast pass).
    bool fused = T == 1 && act_dtype == MDBF_BF16 && P <= kMaxSiblings;
    for (int p = 0; p < P && fused; ++p) {
        const Layer &L = terms[p]->L;
        fused = L.d.env_dtype != MDBF_F32 && L.d.l <= 32 && L.vxA && L.vxB && L.LP == terms[0]->L.LP &&
                terms[p]->kernel == MDBF_KERNEL_AUTO && tmem_path_supports(L, 1);
    }
    if (fused) {
        Layer *Ls[kMaxSiblings];
        for (int p = 0; p < P; ++p) {
            Ls[p] = &terms[p]->L;
            Ls[p]->out_mode = 0;
            Ls[p]->last_ksplit = 0;
            terms[p]->last_kernel = MDBF_KERNEL_TMEM;
            terms[p]->last_launches = 0;
        }
        mdbf_status_t rc = launch_forward_tmem_t1_sum(Ls, P, x, acc, y, st);
        if (rc) return rc;
        terms[0]->last_launches = last_t1_launch_count();
        return MDBF_OK;
    }
    // otherwise: term 0 stores its fp32 output into acc, the others add to it (stream order), a cast pass follows
    for (int p = 0; p < P; ++p) {
        mdbf_status_t rc = forward_impl(terms[p], x, acc, T, act_dtype, st, p == 0 ? 1 : 2);
        if (rc) return rc;
    }
    return launch_cast(acc, y, (size_t)T * terms[0]->L.d.d_out, act_dtype, st);
}

mdbf_status_t mdbf_linear_forward_siblings(const mdbf_handle_t *layers, int32_t n, const void *x, void *const *ys,
                                           int32_t T, int32_t act_dtype, void *stream) {
    if (!layers || !x || !ys) { set_error("mdbf_linear_forward_siblings: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    if (n < 1 || n > 64) { set_error("mdbf_linear_forward_siblings: n=%d outside [1, 64]", n); return MDBF_ERR_SHAPE; }
    bool fusable = T == 1 && act_dtype == MDBF_BF16;
    const int32_t k0 = layers[0] ? layers[0]->kernel : 0;       // checked below; AUTO, or the same one-token kernel forced on every layer
    for (int i = 0; i < n; ++i) {
        mdbf_status_t rc = check_handle(layers[i], "mdbf_linear_forward_siblings");
        if (rc) return rc;
        if (!ys[i]) { set_error("mdbf_linear_forward_siblings: NULL output %d", i); return MDBF_ERR_INVALID_ARG; }
        const Layer &L = layers[i]->L;
        rc = check_device(L, "mdbf_linear_forward_siblings");
        if (rc) return rc;
        if (L.d.d_in != layers[0]->L.d.d_in) {
            set_error("mdbf_linear_forward_siblings: layer %d has d_in=%d, layer 0 has %d", i, L.d.d_in, layers[0]->L.d.d_in);
            return MDBF_ERR_SHAPE;
        }
        if (T < 1 || T > L.d.max_T) {
            set_error("mdbf_linear_forward_siblings: T=%d outside [1, max_T=%d] of layer %d", T, L.d.max_T, i);
            return MDBF_ERR_SHAPE;
        }
        for (int q = 0; q < i; ++q)
            if (layers[q] == layers[i]) { set_error("mdbf_linear_forward_siblings: layer %d repeats layer %d", i, q); return MDBF_ERR_INVALID_ARG; }
        fusable = fusable && L.vxA && L.vxB && L.LP == layers[0]->L.LP && layers[i]->kernel == k0 &&
                  (k0 == MDBF_KERNEL_AUTO || k0 == MDBF_KERNEL_TMEM || k0 == MDBF_KERNEL_I8);
    }
    if (!valid_dtype(act_dtype)) { set_error("mdbf_linear_forward_siblings: bad act_dtype %d", act_dtype); return MDBF_ERR_DTYPE; }
    cudaStream_t st = (cudaStream_t)stream;
    if (!fusable) {                          // more than one token, mixed envelope ranks, fp32 layers: one after the other
        for (int i = 0; i < n; ++i) {
            mdbf_status_t rc = forward_impl(layers[i], x, ys[i], T, act_dtype, st);
            if (rc) return rc;
        }
        return MDBF_OK;
    }
    for (int i0 = 0; i0 < n; i0 += kMaxSiblings) {      // groups of up to kMaxSiblings layers per set of launches
        const int m = n - i0 < kMaxSiblings ? n - i0 : kMaxSiblings;
        Layer *Ls[kMaxSiblings];
        void *outs[kMaxSiblings];
        for (int i = 0; i < m; ++i) {
            Ls[i] = &layers[i0 + i]->L;
            Ls[i]->out_mode = 0;
            Ls[i]->last_ksplit = 0;
            outs[i] = ys[i0 + i];
        }
        int launches = 0, used = 0;
        mdbf_status_t rc = forward_t1_auto(Ls, m, x, outs, st, k0 == MDBF_KERNEL_I8 ? 2 : k0 == MDBF_KERNEL_TMEM ? 1 : 0, &launches, &used);
        if (rc) return rc;
        for (int i = 0; i < m; ++i) {
            layers[i0 + i]->last_launches = i == 0 ? launches : 0;
            layers[i0 + i]->last_kernel = used;
        }
    }
    return MDBF_OK;
}

static mdbf_status_t forward_host_impl(mdbf_handle_t h, const void *x_host, void *y_host, int32_t T, int32_t act_dtype, void *stream,
                                       bool wait) {
    mdbf_status_t rc = check_handle(h, "mdbf_linear_forward_host");
    if (rc) return rc;
    if (!x_host || !y_host) { set_error("mdbf_linear_forward_host: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    Layer &L = h->L;
    if (T < 1 || T > L.d.max_T) {
        set_error("mdbf_linear_forward_host: T=%d outside [1, max_T=%d]", T, L.d.max_T);
        return MDBF_ERR_SHAPE;
    }
    if (!valid_dtype(act_dtype)) { set_error("mdbf_linear_forward_host: bad act_dtype %d", act_dtype); return MDBF_ERR_DTYPE; }
    cudaStream_t st = (cudaStream_t)stream;
    const size_t es = dtype_size(act_dtype);
    if (!L.xstage) {
        set_error("mdbf_linear_forward_host: no staging buffers on this handle; call mdbf_prepare_host_staging(handle) once first (it allocates)");
        return MDBF_ERR_INVALID_ARG;
    }
    MDBF_CUDA(cudaMemcpyAsync(L.xstage, x_host, (size_t)T * L.d.d_in * es, cudaMemcpyHostToDevice, st));
    rc = forward_impl(h, L.xstage, L.ystage, T, act_dtype, st);
    if (rc) return rc;
    MDBF_CUDA(cudaMemcpyAsync(y_host, L.ystage, (size_t)T * L.d.d_out * es, cudaMemcpyDeviceToHost, st));
    if (wait) MDBF_CUDA(cudaStreamSynchronize(st));
    return MDBF_OK;
}

mdbf_status_t mdbf_linear_forward_host(mdbf_handle_t h, const void *x_host, void *y_host, int32_t T,
                                       int32_t act_dtype, void *stream) {
    return forward_host_impl(h, x_host, y_host, T, act_dtype, stream, true);
}

mdbf_status_t mdbf_linear_forward_host_async(mdbf_handle_t h, const void *x_host, void *y_host, int32_t T,
                                             int32_t act_dtype, void *stream) {
    return forward_host_impl(h, x_host, y_host, T, act_dtype, stream, false);
}

mdbf_status_t mdbf_linear_forward_group(const mdbf_handle_t *layers, int32_t n, const void *const *xs, void *const *ys,
                                        int32_t T, int32_t act_dtype, void *stream) {
    if (!layers || !xs || !ys) { set_error("mdbf_linear_forward_group: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    if (n < 1 || n > 64) { set_error("mdbf_linear_forward_group: n=%d outside [1, 64]", n); return MDBF_ERR_SHAPE; }
    if (!valid_dtype(act_dtype)) { set_error("mdbf_linear_forward_group: bad act_dtype %d", act_dtype); return MDBF_ERR_DTYPE; }
    bool fusable = T == 1 && act_dtype == MDBF_BF16;
    for (int i = 0; i < n; ++i) {
        mdbf_status_t rc = check_handle(layers[i], "mdbf_linear_forward_group");
        if (rc) return rc;
        if (!xs[i] || !ys[i]) { set_error("mdbf_linear_forward_group: NULL input or output %d", i); return MDBF_ERR_INVALID_ARG; }
        const Layer &L = layers[i]->L;
        rc = check_device(L, "mdbf_linear_forward_group");
        if (rc) return rc;
        if (T < 1 || T > L.d.max_T) {
            set_error("mdbf_linear_forward_group: T=%d outside [1, max_T=%d] of layer %d", T, L.d.max_T, i);
            return MDBF_ERR_SHAPE;
        }
        for (int q = 0; q < i; ++q)
            if (layers[q] == layers[i]) { set_error("mdbf_linear_forward_group: layer %d repeats layer %d", i, q); return MDBF_ERR_INVALID_ARG; }
        fusable = fusable && t1_supports(L) && L.LP == layers[0]->L.LP &&
                  (layers[i]->kernel == MDBF_KERNEL_AUTO || layers[i]->kernel == MDBF_KERNEL_I8);
    }
    cudaStream_t st = (cudaStream_t)stream;
    if (!fusable || n == 1) {
        for (int i = 0; i < n; ++i) {
            mdbf_status_t rc = forward_impl(layers[i], xs[i], ys[i], T, act_dtype, st);
            if (rc) return rc;
        }
        return MDBF_OK;
    }
    for (int i0 = 0; i0 < n; i0 += 8) {                  // up to eight layers per set of four launches
        const int m = n - i0 < 8 ? n - i0 : 8;
        Layer *Ls[8];
        for (int i = 0; i < m; ++i) {
            Ls[i] = &layers[i0 + i]->L;
            Ls[i]->out_mode = 0;
            Ls[i]->last_ksplit = 0;
            layers[i0 + i]->last_launches = i == 0 ? 4 : 0;
            layers[i0 + i]->last_kernel = MDBF_KERNEL_I8;
        }
        mdbf_status_t rc = launch_forward_t1_group(Ls, m, xs + i0, ys + i0, st, 3);
        if (rc) return rc;
    }
    return MDBF_OK;
}

mdbf_status_t mdbf_prepare_host_staging(mdbf_handle_t h) {
    mdbf_status_t rc = check_handle(h, "mdbf_prepare_host_staging");
    if (rc) return rc;
    rc = check_device(h->L, "mdbf_prepare_host_staging");
    if (rc) return rc;
    return ensure_host_staging(h->L);
}

mdbf_status_t mdbf_get_intermediate(mdbf_handle_t h, float *z, int32_t T, int out_on_device, void *stream) {
    mdbf_status_t rc = check_handle(h, "mdbf_get_intermediate");
    if (rc) return rc;
    Layer &L = h->L;
    if (!z) { set_error("mdbf_get_intermediate: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    if (T < 1 || T > L.d.max_T) { set_error("mdbf_get_intermediate: bad T"); return MDBF_ERR_SHAPE; }
    cudaStream_t st = (cudaStream_t)stream;
    rc = launch_zsum(L, T, st);
    if (rc) return rc;
    MDBF_CUDA(cudaMemcpyAsync(z, L.zsum, (size_t)T * L.d.k * sizeof(float),
                              out_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost, st));
    MDBF_CUDA(cudaStreamSynchronize(st));
    return MDBF_OK;
}

mdbf_status_t mdbf_reconstruct(mdbf_handle_t h, float *W, void *stream) {
    mdbf_status_t rc = check_handle(h, "mdbf_reconstruct");
    if (rc) return rc;
    if (!W) { set_error("mdbf_reconstruct: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    return launch_reconstruct(h->L, W, (cudaStream_t)stream);
}

mdbf_status_t mdbf_poll_status(mdbf_handle_t h, int32_t *device_status) {
    mdbf_status_t rc = check_handle(h, "mdbf_poll_status");
    if (rc) return rc;
    if (!device_status) { set_error("mdbf_poll_status: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    MDBF_CUDA(cudaDeviceSynchronize());
    MDBF_CUDA(cudaMemcpy(device_status, h->L.status, sizeof(int32_t), cudaMemcpyDeviceToHost));
    MDBF_CUDA(cudaMemset(h->L.status, 0, sizeof(int32_t)));
    return MDBF_OK;
}

mdbf_status_t mdbf_selftest_wait_timeout(mdbf_handle_t h, void *stream) {
    mdbf_status_t rc = check_handle(h, "mdbf_selftest_wait_timeout");
    if (rc) return rc;
    return launch_wait_timeout_selftest(h->L, (cudaStream_t)stream);
}

mdbf_status_t mdbf_last_launch_count(mdbf_handle_t h, int32_t *count) {
    mdbf_status_t rc = check_handle(h, "mdbf_last_launch_count");
    if (rc) return rc;
    if (!count) { set_error("mdbf_last_launch_count: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    *count = h->last_launches;
    return MDBF_OK;
}

mdbf_status_t mdbf_last_kernel(mdbf_handle_t h, int32_t *kernel) {
    mdbf_status_t rc = check_handle(h, "mdbf_last_kernel");
    if (rc) return rc;
    if (!kernel) { set_error("mdbf_last_kernel: NULL pointer"); return MDBF_ERR_INVALID_ARG; }
    *kernel = h->last_kernel;
    return MDBF_OK;
}

mdbf_status_t mdbf_destroy(mdbf_handle_t h) {
    mdbf_status_t rc = check_handle(h, "mdbf_destroy");
    if (rc) return rc;
    cudaDeviceSynchronize();
    free_layer(h->L);
    h->magic = 0;
    delete h;
    return MDBF_OK;
}

}  // extern "C"
