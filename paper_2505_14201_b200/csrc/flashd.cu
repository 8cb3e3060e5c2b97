// C ABI of the FLASH-D attention library (see include/flashd.h): argument
// validation, tensor-map construction and kernel launches.  One translation
// unit: the kernels are included as headers.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <mutex>

#include "flashd.h"
#include "flashd_common.cuh"
#include "flashd_decode.cuh"
#include "flashd_perkey.cuh"
#include "flashd_prefill.cuh"
#include "flashd_gqa.cuh"
#include "flashd_pwl.cuh"
#include "flashd_skipstats.cuh"

namespace {

using namespace flashd;

std::atomic<long long> g_launches{0};

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_common(const void* q, const void* k, const void* v, const void* o, int B, int H, int Nq, int Nk,
                 int d, float scale) {
    if (!q || !k || !v || !o) return FLASHD_ERR_NULL;
    if (B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0 || d <= 0 || !std::isfinite(scale)) return FLASHD_ERR_SHAPE;
    if ((long long)B * H > 0x7fffffffLL / 2) return FLASHD_ERR_SHAPE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return FLASHD_ERR_ALIGN;
    return FLASHD_OK;
}

int after_launch() {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? FLASHD_OK : FLASHD_ERR_CUDA;
}

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev] = n;
    }
    return cached[dev];
}

// ----------------------------------------------------------------- tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// [BH, N, D] tensor of bf16 (eb = 2) or one-byte E4M3 (eb = 1) elements, box = 128 bytes of
// columns x 128 rows x 1 head, 128-byte swizzle, rows outside [0, N) read as zero.
bool make_map(CUtensorMap* map, const void* base, int BH, int N, int D, int eb = 2) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)N, (cuuint64_t)BH};
    const cuuint64_t strides[2] = {(cuuint64_t)D * eb, (cuuint64_t)N * D * eb};
    const cuuint32_t box[3] = {(cuuint32_t)(128 / eb), 128, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, eb == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 3,
              const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int EB = 2>
int launch_prefill(const void* q, const void* k, const void* v, void* o, float* lse, int out_f32, int BH, int Nq,
                   int Nk, float scale, int causal, cudaStream_t stream) {
    using C = PrefillCfg<D, EB>;
    CUtensorMap mq, mk, mv;
    if (!make_map(&mq, q, BH, Nq, D, EB) || !make_map(&mk, k, BH, Nk, D, EB) || !make_map(&mv, v, BH, Nk, D, EB))
        return FLASHD_ERR_CUDA;
    static bool attr_set[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FLASHD_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(prefill_kernel<D, EB>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) !=
            cudaSuccess)
            return FLASHD_ERR_CUDA;
        attr_set[dev] = true;
    }
    PrefillParams prm;
    prm.o = o;
    prm.lse = lse;
    prm.BH = BH;
    prm.Nq = Nq;
    prm.Nk = Nk;
    prm.scale_log2e = scale * kLog2e;
    prm.causal = causal ? 1 : 0;
    prm.out_f32 = out_f32;
    prm.n_qpairs = (Nq + C::kItemRows - 1) / C::kItemRows;
    prm.n_work = BH * prm.n_qpairs;
    const int sms = sm_count();
    if (sms <= 0) return FLASHD_ERR_CUDA;
    const int grid = prm.n_work < sms ? prm.n_work : sms;
    // launched with programmatic stream serialisation: the grid may be set up while the previous
    // kernel of the stream drains (the kernel itself waits for that kernel before it reads or writes
    // global memory)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)C::kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, prefill_kernel<D, EB>, mq, mk, mv, prm) != cudaSuccess) {
        g_launches.fetch_add(1, std::memory_order_relaxed);
        cudaGetLastError();
        return FLASHD_ERR_CUDA;
    }
    return after_launch();
}

template <typename TIn, typename TOut>
int launch_perkey_t(const void* q, const void* k, const void* v, void* o, float* lse, long long rows, int Nq,
                    int Nk, int d, float scale, int causal, cudaStream_t stream) {
    const int warps = 4;
    const long long blocks = (rows + warps - 1) / warps;
    if (blocks > 0x7fffffffLL) return FLASHD_ERR_SHAPE;
    const TIn* qq = static_cast<const TIn*>(q);
    const TIn* kk = static_cast<const TIn*>(k);
    const TIn* vv = static_cast<const TIn*>(v);
    TOut* oo = static_cast<TOut*>(o);
    switch (d) {
        case 16:
        case 32: perkey_kernel<TIn, TOut, 1><<<(unsigned)blocks, warps * 32, 0, stream>>>(qq, kk, vv, oo, lse, rows, Nq, Nk, scale, causal, d); break;
        case 64: perkey_kernel<TIn, TOut, 2><<<(unsigned)blocks, warps * 32, 0, stream>>>(qq, kk, vv, oo, lse, rows, Nq, Nk, scale, causal, d); break;
        case 128: perkey_kernel<TIn, TOut, 4><<<(unsigned)blocks, warps * 32, 0, stream>>>(qq, kk, vv, oo, lse, rows, Nq, Nk, scale, causal, d); break;
        case 256: perkey_kernel<TIn, TOut, 8><<<(unsigned)blocks, warps * 32, 0, stream>>>(qq, kk, vv, oo, lse, rows, Nq, Nk, scale, causal, d); break;
        default: return FLASHD_ERR_UNSUPPORTED;
    }
    return after_launch();
}

template <typename TIn, typename TOut>
int launch_pwl_t(const void* q, const void* k, const void* v, void* o, unsigned long long* counts, long long rows,
                 int Nq, int Nk, int d, float scale, int causal, const PwlTables& tab, float lo, float hi,
                 int range_mode, cudaStream_t stream) {
    const int warps = 4;
    const long long blocks = (rows + warps - 1) / warps;
    if (blocks > 0x7fffffffLL) return FLASHD_ERR_SHAPE;
    const TIn* qq = static_cast<const TIn*>(q);
    const TIn* kk = static_cast<const TIn*>(k);
    const TIn* vv = static_cast<const TIn*>(v);
    TOut* oo = static_cast<TOut*>(o);
    const unsigned g = (unsigned)blocks;
    switch (d) {
        case 16:
        case 32: perkey_pwl_kernel<TIn, TOut, 1><<<g, warps * 32, 0, stream>>>(qq, kk, vv, oo, counts, rows, Nq, Nk, scale, causal, tab, lo, hi, range_mode, d); break;
        case 64: perkey_pwl_kernel<TIn, TOut, 2><<<g, warps * 32, 0, stream>>>(qq, kk, vv, oo, counts, rows, Nq, Nk, scale, causal, tab, lo, hi, range_mode, d); break;
        case 128: perkey_pwl_kernel<TIn, TOut, 4><<<g, warps * 32, 0, stream>>>(qq, kk, vv, oo, counts, rows, Nq, Nk, scale, causal, tab, lo, hi, range_mode, d); break;
        case 256: perkey_pwl_kernel<TIn, TOut, 8><<<g, warps * 32, 0, stream>>>(qq, kk, vv, oo, counts, rows, Nq, Nk, scale, causal, tab, lo, hi, range_mode, d); break;
        default: return FLASHD_ERR_UNSUPPORTED;
    }
    return after_launch();
}

// copies one host table into the kernel-parameter block; false if malformed
bool fill_table(int n, const float* x, const float* y, int* n_out, float* xs, float* ys) {
    for (int t = 0; t <= FLASHD_PWL_MAX_SEGMENTS; ++t) { xs[t] = 0.f; ys[t] = 0.f; }
    *n_out = 0;
    if (n == 0) return true;
    if (n < 0 || n > FLASHD_PWL_MAX_SEGMENTS || !x || !y) return false;
    for (int t = 0; t <= n; ++t) {
        if (!std::isfinite(x[t]) || !std::isfinite(y[t])) return false;
        if (t > 0 && !(x[t] > x[t - 1])) return false;
        xs[t] = x[t];
        ys[t] = y[t];
    }
    *n_out = n;
    return true;
}

template <int D, int KVB = 2, bool PAGED = false>
int launch_partial(const void* q, const void* k, const void* v, void* ws, long long rows, int Nq, int Nk,
                   float scale, int num_splits, cudaStream_t stream, const PagedKV& pg = PagedKV{}) {
    using C = DecodeCfg<D, KVB>;
    static bool attr_set[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FLASHD_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(splitk_partial_kernel<D, KVB, PAGED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 C::kSmemBytes) != cudaSuccess)
            return FLASHD_ERR_CUDA;
        attr_set[dev] = true;
    }
    const int sms = sm_count();
    if (sms <= 0) return FLASHD_ERR_CUDA;
    const long long items = rows * num_splits;
    const int grid = (int)(items < sms ? items : sms);
    splitk_partial_kernel<D, KVB, PAGED><<<grid, C::kThreads, C::kSmemBytes, stream>>>(
        static_cast<const __nv_bfloat16*>(q), static_cast<const unsigned char*>(k),
        static_cast<const unsigned char*>(v), static_cast<float*>(ws), rows, Nq, Nk, scale * kLog2e, num_splits, pg);
    return after_launch();
}

template <int D, bool PAGED = false>
int launch_gqa_partial(const void* q, const void* k, const void* v, void* ws, int BHkv, int R, int Nq, int causal,
                       int Nk, float scale, int num_splits, cudaStream_t stream, const PagedKV& pg = PagedKV{}) {
    using C = GqaCfg<D>;
    CUtensorMap mk, mv;
    // contiguous: (D, Nk, B*Hkv); paged: the pool as (D, page_size, num_pages*Hkv)
    const int slabs = PAGED ? pg.num_pages * pg.H : BHkv;
    const int rows_per_slab = PAGED ? pg.page_size : Nk;
    if (!make_map(&mk, k, slabs, rows_per_slab, D) || !make_map(&mv, v, slabs, rows_per_slab, D)) return FLASHD_ERR_CUDA;
    static bool attr_set[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FLASHD_ERR_CUDA;
    if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(gqa_partial_kernel<D, PAGED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 C::kSmemBytes) != cudaSuccess)
            return FLASHD_ERR_CUDA;
        attr_set[dev] = true;
    }
    const int sms = sm_count();
    if (sms <= 0) return FLASHD_ERR_CUDA;
    const long long items = (long long)BHkv * num_splits;
    const int grid = (int)(items < sms ? items : sms);
    gqa_partial_kernel<D, PAGED><<<grid, C::kThreads, C::kSmemBytes, stream>>>(
        mk, mv, static_cast<const __nv_bfloat16*>(q), static_cast<float*>(ws), BHkv, R, Nq, causal, Nk,
        scale * kLog2e, num_splits, pg);
    return after_launch();
}

// Scratch of the allocation-free split-K entry point: partial states
// [rows, splits, d+1] fp32.  Part of the library image, so every device that
// loads the library holds it until exit.  In host code this name is only a
// handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) float g_static_scratch[FLASHD_STATIC_SCRATCH_BYTES / sizeof(float)];

// Device address of g_static_scratch on the current device, looked up once per
// device; nullptr if the lookup failed.
float* static_scratch_ptr() {
    static std::mutex mu;
    static float* cached[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev] == nullptr) {
        float* ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch) != cudaSuccess) return nullptr;
        cached[dev] = ptr;
    }
    return cached[dev];
}

int check_splits(int Nk, int num_splits) {
    if (num_splits < 1 || num_splits > FLASHD_MAX_SPLITS || num_splits > Nk) return FLASHD_ERR_WORKSPACE;
    // every split but the last must be non-empty by construction; the last one is
    // non-empty iff (S-1)*ceil(Nk/S) < Nk, otherwise it is written as empty (L = -inf)
    return FLASHD_OK;
}

}  // namespace

// ============================================================================ C ABI
// Per-device helper streams and events of the host entry point (created on first use).
namespace {
struct HostPipe {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_out = nullptr;
    cudaEvent_t ev_in[16] = {nullptr}, ev_k[16] = {nullptr};
};
HostPipe g_pipe[64];
std::mutex g_pipe_mutex;

bool host_pipe_init(HostPipe& hp) {
    if (hp.ready) return true;
    bool ok = cudaStreamCreateWithFlags(&hp.s_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&hp.s_out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.ev_start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&hp.ev_out, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < 16; ++i)
        ok = cudaEventCreateWithFlags(&hp.ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&hp.ev_k[i], cudaEventDisableTiming) == cudaSuccess;
    hp.ready = ok;
    return ok;
}
}  // namespace

extern "C" {

int flashd_version(void) { return 100; }

long long flashd_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* flashd_status_string(int status) {
    switch (status) {
        case FLASHD_OK: return "ok";
        case FLASHD_ERR_NULL: return "null pointer";
        case FLASHD_ERR_SHAPE: return "invalid size or scale";
        case FLASHD_ERR_UNSUPPORTED: return "unsupported head size, dtype or mode";
        case FLASHD_ERR_ALIGN: return "pointer not 16-byte aligned";
        case FLASHD_ERR_WORKSPACE: return "workspace too small or bad split count";
        case FLASHD_ERR_CUDA: return "CUDA call failed";
        case FLASHD_ERR_TIMEOUT: return "bounded wait inside a kernel ran out";
        default: return "unknown status";
    }
}

int flashd_attn_fwd_ex(const void* q, const void* k, const void* v, void* o, float* lse_out, int in_dtype,
                       int out_dtype, int B, int H, int Nq, int Nk, int d, float scale, int causal, void* stream) {
    const int st = check_common(q, k, v, o, B, H, Nq, Nk, d, scale);
    if (st != FLASHD_OK) return st;
    if (in_dtype != FLASHD_BF16 || (out_dtype != FLASHD_BF16 && out_dtype != FLASHD_F32)) return FLASHD_ERR_UNSUPPORTED;
    if (scale == 0.f) return FLASHD_ERR_UNSUPPORTED;
    if (o == q || o == k || o == v) return FLASHD_ERR_SHAPE;
    const int BH = B * H;
    if (d == 128) return launch_prefill<128>(q, k, v, o, lse_out, out_dtype == FLASHD_F32, BH, Nq, Nk, scale, causal, as_stream(stream));
    if (d == 64) return launch_prefill<64>(q, k, v, o, lse_out, out_dtype == FLASHD_F32, BH, Nq, Nk, scale, causal, as_stream(stream));
    if (d == 256) return launch_prefill<256>(q, k, v, o, lse_out, out_dtype == FLASHD_F32, BH, Nq, Nk, scale, causal, as_stream(stream));
    return FLASHD_ERR_UNSUPPORTED;
}

int flashd_attn_fwd_fp8(const void* q, const void* k, const void* v, void* o, float* lse_out, int out_dtype, int B,
                        int H, int Nq, int Nk, int d, float scale, int causal, void* stream) {
    const int st = check_common(q, k, v, o, B, H, Nq, Nk, d, scale);
    if (st != FLASHD_OK) return st;
    if (out_dtype != FLASHD_BF16 && out_dtype != FLASHD_F32) return FLASHD_ERR_UNSUPPORTED;
    if ((d != 128 && d != 256) || scale == 0.f) return FLASHD_ERR_UNSUPPORTED;
    if (o == q || o == k || o == v) return FLASHD_ERR_SHAPE;
    if (d == 256)
        return launch_prefill<256, 1>(q, k, v, o, lse_out, out_dtype == FLASHD_F32, B * H, Nq, Nk, scale, causal,
                                      as_stream(stream));
    return launch_prefill<128, 1>(q, k, v, o, lse_out, out_dtype == FLASHD_F32, B * H, Nq, Nk, scale, causal,
                                  as_stream(stream));
}

int flashd_attn_fwd(const void* q, const void* k, const void* v, void* o, int B, int H, int Nq, int Nk, int d,
                    float scale, int causal, void* stream) {
    return flashd_attn_fwd_ex(q, k, v, o, nullptr, FLASHD_BF16, FLASHD_BF16, B, H, Nq, Nk, d, scale, causal, stream);
}

int flashd_attn_fwd_perkey(const void* q, const void* k, const void* v, void* o, float* lse_out, int in_dtype,
                           int out_dtype, int B, int H, int Nq, int Nk, int d, float scale, int causal,
                           void* stream) {
    const int st = check_common(q, k, v, o, B, H, Nq, Nk, d, scale);
    if (st != FLASHD_OK) return st;
    if (d != 16 && d != 32 && d != 64 && d != 128 && d != 256) return FLASHD_ERR_UNSUPPORTED;
    const long long rows = (long long)B * H * Nq;
    cudaStream_t s = as_stream(stream);
    if (in_dtype == FLASHD_F32 && out_dtype == FLASHD_F32)
        return launch_perkey_t<float, float>(q, k, v, o, lse_out, rows, Nq, Nk, d, scale, causal, s);
    if (in_dtype == FLASHD_BF16 && out_dtype == FLASHD_BF16)
        return launch_perkey_t<__nv_bfloat16, __nv_bfloat16>(q, k, v, o, lse_out, rows, Nq, Nk, d, scale, causal, s);
    if (in_dtype == FLASHD_BF16 && out_dtype == FLASHD_F32)
        return launch_perkey_t<__nv_bfloat16, float>(q, k, v, o, lse_out, rows, Nq, Nk, d, scale, causal, s);
    return FLASHD_ERR_UNSUPPORTED;
}

int flashd_attn_fwd_pwl(const void* q, const void* k, const void* v, void* o, unsigned long long* counts,
                        int in_dtype, int out_dtype, int B, int H, int Nq, int Nk, int d, float scale, int causal,
                        int sig_n, const float* sig_x, const float* sig_y, int ln_n, const float* ln_x,
                        const float* ln_y, float lo, float hi, int range_mode, void* stream) {
    const int st = check_common(q, k, v, o, B, H, Nq, Nk, d, scale);
    if (st != FLASHD_OK) return st;
    if (d != 16 && d != 32 && d != 64 && d != 128 && d != 256) return FLASHD_ERR_UNSUPPORTED;
    if (range_mode != 0 && range_mode != 1) return FLASHD_ERR_SHAPE;
    if (std::isnan(lo) || std::isnan(hi) || !(lo <= hi)) return FLASHD_ERR_SHAPE;
    PwlTables tab;
    if (!fill_table(sig_n, sig_x, sig_y, &tab.sig_n, tab.sig_x, tab.sig_y)) return FLASHD_ERR_SHAPE;
    if (!fill_table(ln_n, ln_x, ln_y, &tab.ln_n, tab.ln_x, tab.ln_y)) return FLASHD_ERR_SHAPE;
    const long long rows = (long long)B * H * Nq;
    cudaStream_t s = as_stream(stream);
    if (in_dtype == FLASHD_F32 && out_dtype == FLASHD_F32)
        return launch_pwl_t<float, float>(q, k, v, o, counts, rows, Nq, Nk, d, scale, causal, tab, lo, hi, range_mode, s);
    if (in_dtype == FLASHD_BF16 && out_dtype == FLASHD_BF16)
        return launch_pwl_t<__nv_bfloat16, __nv_bfloat16>(q, k, v, o, counts, rows, Nq, Nk, d, scale, causal, tab, lo, hi, range_mode, s);
    if (in_dtype == FLASHD_BF16 && out_dtype == FLASHD_F32)
        return launch_pwl_t<__nv_bfloat16, float>(q, k, v, o, counts, rows, Nq, Nk, d, scale, causal, tab, lo, hi, range_mode, s);
    return FLASHD_ERR_UNSUPPORTED;
}

int flashd_attn_fwd_f32(const void* q, const void* k, const void* v, void* o, int B, int H, int Nq, int Nk, int d,
                        float scale, int causal, void* stream) {
    return flashd_attn_fwd_perkey(q, k, v, o, nullptr, FLASHD_F32, FLASHD_F32, B, H, Nq, Nk, d, scale, causal, stream);
}

size_t flashd_splitk_workspace_bytes(int B, int H, int Nq, int d, int num_splits) {
    if (B <= 0 || H <= 0 || Nq <= 0 || d <= 0 || num_splits <= 0) return 0;
    return (size_t)B * H * Nq * num_splits * (size_t)(d + 1) * sizeof(float);
}

int flashd_splitk_num_splits(int B, int H, int Nq, int Nk, int d) {
    (void)d;
    if (B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0) return 0;
    const long long rows = (long long)B * H * Nq;
    // enough work items for ~32 waves on a 148-SM part, splits of at least 512 keys
    long long want = (32LL * 148 + rows - 1) / rows;
    int s = 1;
    while (s < want && s < FLASHD_MAX_SPLITS) s *= 2;
    if (Nk >= 8192 && s < 2) s = 2;
    while (s > 1 && Nk / s < 512) s /= 2;
    return s;
}

int flashd_splitk_partial(const void* q, const void* k, const void* v, void* workspace, size_t workspace_bytes,
                          int B, int H, int Nq, int Nk, int d, float scale, int num_splits, void* stream) {
    const int st = check_common(q, k, v, workspace, B, H, Nq, Nk, d, scale);
    if (st != FLASHD_OK) return st;
    if (d != 128 && d != 64) return FLASHD_ERR_UNSUPPORTED;
    const int cs = check_splits(Nk, num_splits);
    if (cs != FLASHD_OK) return cs;
    if (workspace_bytes < flashd_splitk_workspace_bytes(B, H, Nq, d, num_splits)) return FLASHD_ERR_WORKSPACE;
    const long long rows = (long long)B * H * Nq;
    if (d == 128) return launch_partial<128>(q, k, v, workspace, rows, Nq, Nk, scale, num_splits, as_stream(stream));
    return launch_partial<64>(q, k, v, workspace, rows, Nq, Nk, scale, num_splits, as_stream(stream));
}

int flashd_splitk_combine(const void* workspace, void* o, float* lse_out, int B, int H, int Nq, int d,
                          int num_splits, int out_dtype, void* stream) {
    if (!workspace || !o) return FLASHD_ERR_NULL;
    if (B <= 0 || H <= 0 || Nq <= 0 || d <= 0) return FLASHD_ERR_SHAPE;
    if (d != 128 && d != 64) return FLASHD_ERR_UNSUPPORTED;
    if (out_dtype != FLASHD_BF16 && out_dtype != FLASHD_F32) return FLASHD_ERR_UNSUPPORTED;
    if (num_splits < 1 || num_splits > FLASHD_MAX_SPLITS) return FLASHD_ERR_WORKSPACE;
    if (!aligned16(workspace) || !aligned16(o)) return FLASHD_ERR_ALIGN;
    const long long rows = (long long)B * H * Nq;
    if (rows > 0x7fffffffLL) return FLASHD_ERR_SHAPE;
    const float* ws = static_cast<const float*>(workspace);
    cudaStream_t s = as_stream(stream);
    if (d == 128) {
        if (out_dtype == FLASHD_F32) splitk_combine_kernel<128, float><<<(unsigned)rows, 128, 0, s>>>(ws, static_cast<float*>(o), lse_out, num_splits);
        else splitk_combine_kernel<128, __nv_bfloat16><<<(unsigned)rows, 128, 0, s>>>(ws, static_cast<__nv_bfloat16*>(o), lse_out, num_splits);
    } else {
        if (out_dtype == FLASHD_F32) splitk_combine_kernel<64, float><<<(unsigned)rows, 64, 0, s>>>(ws, static_cast<float*>(o), lse_out, num_splits);
        else splitk_combine_kernel<64, __nv_bfloat16><<<(unsigned)rows, 64, 0, s>>>(ws, static_cast<__nv_bfloat16*>(o), lse_out, num_splits);
    }
    return after_launch();
}

int flashd_attn_fwd_splitk(const void* q, const void* k, const void* v, void* o, void* workspace,
                           size_t workspace_bytes, int B, int H, int Nq, int Nk, int d, float scale, int num_splits,
                           void* stream) {
    if (!o) return FLASHD_ERR_NULL;
    if (num_splits <= 0) num_splits = flashd_splitk_num_splits(B, H, Nq, Nk, d);
    if (!workspace) return FLASHD_ERR_NULL;
    int st = flashd_splitk_partial(q, k, v, workspace, workspace_bytes, B, H, Nq, Nk, d, scale, num_splits, stream);
    if (st != FLASHD_OK) return st;
    return flashd_splitk_combine(workspace, o, nullptr, B, H, Nq, d, num_splits, FLASHD_BF16, stream);
}

int flashd_splitk_partial_fp8kv(const void* q, const void* k, const void* v, void* workspace, size_t workspace_bytes,
                                int B, int H, int Nq, int Nk, int d, float scale, int num_splits, void* stream) {
    const int st = check_common(q, k, v, workspace, B, H, Nq, Nk, d, scale);
    if (st != FLASHD_OK) return st;
    if (d != 128 && d != 64) return FLASHD_ERR_UNSUPPORTED;
    const int cs = check_splits(Nk, num_splits);
    if (cs != FLASHD_OK) return cs;
    if (workspace_bytes < flashd_splitk_workspace_bytes(B, H, Nq, d, num_splits)) return FLASHD_ERR_WORKSPACE;
    const long long rows = (long long)B * H * Nq;
    if (d == 128) return launch_partial<128, 1>(q, k, v, workspace, rows, Nq, Nk, scale, num_splits, as_stream(stream));
    return launch_partial<64, 1>(q, k, v, workspace, rows, Nq, Nk, scale, num_splits, as_stream(stream));
}

int flashd_attn_fwd_splitk_fp8kv(const void* q, const void* k, const void* v, void* o, void* workspace,
                                 size_t workspace_bytes, int B, int H, int Nq, int Nk, int d, float scale,
                                 int num_splits, void* stream) {
    if (!o || !workspace) return FLASHD_ERR_NULL;
    if (num_splits <= 0) num_splits = flashd_splitk_num_splits(B, H, Nq, Nk, d);
    const int st = flashd_splitk_partial_fp8kv(q, k, v, workspace, workspace_bytes, B, H, Nq, Nk, d, scale,
                                               num_splits, stream);
    if (st != FLASHD_OK) return st;
    return flashd_splitk_combine(workspace, o, nullptr, B, H, Nq, d, num_splits, FLASHD_BF16, stream);
}

static int splitk_partial_paged_impl(int kvb, const void* q, const void* k_pages, const void* v_pages, const int* block_table,
                                const int* seq_lens, void* workspace, size_t workspace_bytes, int B, int H, int Nq,
                                int max_pages, int page_size, int num_pages, int d, float scale, int num_splits,
                                void* stream) {
    if (!q || !k_pages || !v_pages || !block_table || !seq_lens || !workspace) return FLASHD_ERR_NULL;
    if (B <= 0 || H <= 0 || Nq <= 0 || max_pages <= 0 || page_size <= 0 || num_pages <= 0 || d <= 0 ||
        !std::isfinite(scale))
        return FLASHD_ERR_SHAPE;
    if ((long long)B * H > 0x7fffffffLL / 2 || (long long)max_pages * page_size > 0x7fffffffLL) return FLASHD_ERR_SHAPE;
    if (!aligned16(q) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(workspace) ||
        (reinterpret_cast<uintptr_t>(block_table) & 3u) || (reinterpret_cast<uintptr_t>(seq_lens) & 3u))
        return FLASHD_ERR_ALIGN;
    if (d != 128 && d != 64) return FLASHD_ERR_UNSUPPORTED;
    const int chunk = 16384 / (d * kvb);                           // keys per ring stage (DecodeCfg::kChunk)
    if (page_size % chunk != 0) return FLASHD_ERR_UNSUPPORTED;     // a ring stage must not straddle pages
    if (num_splits < 1 || num_splits > FLASHD_MAX_SPLITS) return FLASHD_ERR_WORKSPACE;
    if (workspace_bytes < flashd_splitk_workspace_bytes(B, H, Nq, d, num_splits)) return FLASHD_ERR_WORKSPACE;
    const long long rows = (long long)B * H * Nq;
    if (rows > 0x7fffffffLL) return FLASHD_ERR_SHAPE;
    PagedKV pg;
    pg.block_table = block_table;
    pg.seq_lens = seq_lens;
    pg.max_pages = max_pages;
    pg.page_size = page_size;
    pg.num_pages = num_pages;
    pg.H = H;
    cudaStream_t s = as_stream(stream);
    if (kvb == 2) {
        if (d == 128) return launch_partial<128, 2, true>(q, k_pages, v_pages, workspace, rows, Nq, 0, scale, num_splits, s, pg);
        return launch_partial<64, 2, true>(q, k_pages, v_pages, workspace, rows, Nq, 0, scale, num_splits, s, pg);
    }
    if (d == 128) return launch_partial<128, 1, true>(q, k_pages, v_pages, workspace, rows, Nq, 0, scale, num_splits, s, pg);
    return launch_partial<64, 1, true>(q, k_pages, v_pages, workspace, rows, Nq, 0, scale, num_splits, s, pg);
}

int flashd_splitk_partial_paged(const void* q, const void* k_pages, const void* v_pages, const int* block_table,
                                const int* seq_lens, void* workspace, size_t workspace_bytes, int B, int H, int Nq,
                                int max_pages, int page_size, int num_pages, int d, float scale, int num_splits,
                                void* stream) {
    return splitk_partial_paged_impl(2, q, k_pages, v_pages, block_table, seq_lens, workspace, workspace_bytes, B, H, Nq,
                                     max_pages, page_size, num_pages, d, scale, num_splits, stream);
}

int flashd_splitk_partial_paged_fp8kv(const void* q, const void* k_pages, const void* v_pages, const int* block_table,
                                      const int* seq_lens, void* workspace, size_t workspace_bytes, int B, int H,
                                      int Nq, int max_pages, int page_size, int num_pages, int d, float scale,
                                      int num_splits, void* stream) {
    return splitk_partial_paged_impl(1, q, k_pages, v_pages, block_table, seq_lens, workspace, workspace_bytes, B, H, Nq,
                                     max_pages, page_size, num_pages, d, scale, num_splits, stream);
}

int flashd_attn_fwd_splitk_paged(const void* q, const void* k_pages, const void* v_pages, void* o,
                                 const int* block_table, const int* seq_lens, void* workspace,
                                 size_t workspace_bytes, int B, int H, int Nq, int max_pages, int page_size,
                                 int num_pages, int d, float scale, int num_splits, void* stream) {
    if (!o) return FLASHD_ERR_NULL;
    if (!aligned16(o)) return FLASHD_ERR_ALIGN;
    if (num_splits <= 0 && B > 0 && H > 0 && Nq > 0 && max_pages > 0 && page_size > 0 &&
        (long long)max_pages * page_size <= 0x7fffffffLL)
        num_splits = flashd_splitk_num_splits(B, H, Nq, max_pages * page_size, d);
    const int st = flashd_splitk_partial_paged(q, k_pages, v_pages, block_table, seq_lens, workspace, workspace_bytes,
                                               B, H, Nq, max_pages, page_size, num_pages, d, scale, num_splits, stream);
    if (st != FLASHD_OK) return st;
    return flashd_splitk_combine(workspace, o, nullptr, B, H, Nq, d, num_splits, FLASHD_BF16, stream);
}

int flashd_attn_fwd_splitk_paged_fp8kv(const void* q, const void* k_pages, const void* v_pages, void* o,
                                 const int* block_table, const int* seq_lens, void* workspace,
                                 size_t workspace_bytes, int B, int H, int Nq, int max_pages, int page_size,
                                 int num_pages, int d, float scale, int num_splits, void* stream) {
    if (!o) return FLASHD_ERR_NULL;
    if (!aligned16(o)) return FLASHD_ERR_ALIGN;
    if (num_splits <= 0 && B > 0 && H > 0 && Nq > 0 && max_pages > 0 && page_size > 0 &&
        (long long)max_pages * page_size <= 0x7fffffffLL)
        num_splits = flashd_splitk_num_splits(B, H, Nq, max_pages * page_size, d);
    const int st = flashd_splitk_partial_paged_fp8kv(q, k_pages, v_pages, block_table, seq_lens, workspace, workspace_bytes,
                                               B, H, Nq, max_pages, page_size, num_pages, d, scale, num_splits, stream);
    if (st != FLASHD_OK) return st;
    return flashd_splitk_combine(workspace, o, nullptr, B, H, Nq, d, num_splits, FLASHD_BF16, stream);
}

int flashd_gqa_num_splits(int B, int Hkv, int G, int Nk, int d) {
    (void)G;
    return flashd_splitk_num_splits(B, Hkv, 1, Nk, d);
}

int flashd_gqa_partial(const void* q, const void* k, const void* v, void* workspace, size_t workspace_bytes, int B,
                       int Hkv, int G, int Nq, int Nk, int d, float scale, int causal, int num_splits,
                       void* stream) {
    if (G < 1 || Nq < 1) return FLASHD_ERR_SHAPE;
    if ((long long)G * Nq > FLASHD_MAX_GROUP) return FLASHD_ERR_UNSUPPORTED;
    if (causal && Nq > Nk) return FLASHD_ERR_SHAPE;
    const int st = check_common(q, k, v, workspace, B, Hkv, Nq, Nk, d, scale);
    if (st != FLASHD_OK) return st;
    if (d != 128 && d != 64) return FLASHD_ERR_UNSUPPORTED;
    const int cs = check_splits(Nk, num_splits);
    if (cs != FLASHD_OK) return cs;
    if ((long long)B * Hkv * G > 0x7fffffffLL / FLASHD_MAX_SPLITS) return FLASHD_ERR_SHAPE;
    if (workspace_bytes < flashd_splitk_workspace_bytes(B, Hkv * G, Nq, d, num_splits)) return FLASHD_ERR_WORKSPACE;
    const int BHkv = B * Hkv;
    const int R = G * Nq;
    const int cz = causal ? 1 : 0;
    if (d == 128)
        return launch_gqa_partial<128>(q, k, v, workspace, BHkv, R, Nq, cz, Nk, scale, num_splits, as_stream(stream));
    return launch_gqa_partial<64>(q, k, v, workspace, BHkv, R, Nq, cz, Nk, scale, num_splits, as_stream(stream));
}

int flashd_attn_fwd_gqa(const void* q, const void* k, const void* v, void* o, void* workspace, size_t workspace_bytes,
                        int B, int Hkv, int G, int Nq, int Nk, int d, float scale, int causal, int num_splits,
                        void* stream) {
    if (!o || !workspace) return FLASHD_ERR_NULL;
    if (num_splits <= 0) num_splits = flashd_gqa_num_splits(B, Hkv, G, Nk, d);
    const int st = flashd_gqa_partial(q, k, v, workspace, workspace_bytes, B, Hkv, G, Nq, Nk, d, scale, causal,
                                      num_splits, stream);
    if (st != FLASHD_OK) return st;
    return flashd_splitk_combine(workspace, o, nullptr, B, Hkv * G, Nq, d, num_splits, FLASHD_BF16, stream);
}

int flashd_gqa_partial_paged(const void* q, const void* k_pages, const void* v_pages, const int* block_table,
                             const int* seq_lens, void* workspace, size_t workspace_bytes, int B, int Hkv, int G,
                             int Nq, int max_pages, int page_size, int num_pages, int d, float scale, int causal,
                             int num_splits, void* stream) {
    if (!q || !k_pages || !v_pages || !block_table || !seq_lens || !workspace) return FLASHD_ERR_NULL;
    if (B <= 0 || Hkv <= 0 || G < 1 || Nq < 1 || max_pages <= 0 || page_size <= 0 || num_pages <= 0 || d <= 0 ||
        !std::isfinite(scale))
        return FLASHD_ERR_SHAPE;
    if ((long long)G * Nq > FLASHD_MAX_GROUP) return FLASHD_ERR_UNSUPPORTED;
    if ((long long)max_pages * page_size > 0x7fffffffLL || (long long)num_pages * Hkv > 0x7fffffffLL) return FLASHD_ERR_SHAPE;
    if ((long long)B * Hkv * G > 0x7fffffffLL / FLASHD_MAX_SPLITS) return FLASHD_ERR_SHAPE;
    if (!aligned16(q) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(workspace) ||
        (reinterpret_cast<uintptr_t>(block_table) & 3u) || (reinterpret_cast<uintptr_t>(seq_lens) & 3u))
        return FLASHD_ERR_ALIGN;
    if (d != 128 && d != 64) return FLASHD_ERR_UNSUPPORTED;
    if (page_size % 128 != 0) return FLASHD_ERR_UNSUPPORTED;        // a 128-key chunk must not straddle pages
    if (num_splits < 1 || num_splits > FLASHD_MAX_SPLITS) return FLASHD_ERR_WORKSPACE;
    if (workspace_bytes < flashd_splitk_workspace_bytes(B, Hkv * G, Nq, d, num_splits)) return FLASHD_ERR_WORKSPACE;
    PagedKV pg;
    pg.block_table = block_table;
    pg.seq_lens = seq_lens;
    pg.max_pages = max_pages;
    pg.page_size = page_size;
    pg.num_pages = num_pages;
    pg.H = Hkv;
    const int cz = causal ? 1 : 0;
    if (d == 128)
        return launch_gqa_partial<128, true>(q, k_pages, v_pages, workspace, B * Hkv, G * Nq, Nq, cz, 0, scale, num_splits,
                                             as_stream(stream), pg);
    return launch_gqa_partial<64, true>(q, k_pages, v_pages, workspace, B * Hkv, G * Nq, Nq, cz, 0, scale, num_splits,
                                        as_stream(stream), pg);
}

int flashd_attn_fwd_gqa_paged(const void* q, const void* k_pages, const void* v_pages, void* o,
                              const int* block_table, const int* seq_lens, void* workspace, size_t workspace_bytes,
                              int B, int Hkv, int G, int Nq, int max_pages, int page_size, int num_pages, int d,
                              float scale, int causal, int num_splits, void* stream) {
    if (!o) return FLASHD_ERR_NULL;
    if (!aligned16(o)) return FLASHD_ERR_ALIGN;
    if (num_splits <= 0 && B > 0 && Hkv > 0 && G > 0 && max_pages > 0 && page_size > 0 &&
        (long long)max_pages * page_size <= 0x7fffffffLL)
        num_splits = flashd_gqa_num_splits(B, Hkv, G, max_pages * page_size, d);
    const int st = flashd_gqa_partial_paged(q, k_pages, v_pages, block_table, seq_lens, workspace, workspace_bytes, B,
                                            Hkv, G, Nq, max_pages, page_size, num_pages, d, scale, causal, num_splits,
                                            stream);
    if (st != FLASHD_OK) return st;
    return flashd_splitk_combine(workspace, o, nullptr, B, Hkv * G, Nq, d, num_splits, FLASHD_BF16, stream);
}

int flashd_attn_fwd_splitk_static(const void* q, const void* k, const void* v, void* o, int B, int H, int Nq,
                                  int Nk, int d, float scale, int num_splits, void* stream) {
    const int st = check_common(q, k, v, o, B, H, Nq, Nk, d, scale);
    if (st != FLASHD_OK) return st;
    if (d != 128 && d != 64) return FLASHD_ERR_UNSUPPORTED;
    if (num_splits <= 0) num_splits = flashd_splitk_num_splits(B, H, Nq, Nk, d);
    const int cs = check_splits(Nk, num_splits);
    if (cs != FLASHD_OK) return cs;
    const long long rows = (long long)B * H * Nq;
    if (rows > 0x7fffffffLL) return FLASHD_ERR_SHAPE;
    const unsigned long long need = (unsigned long long)rows * num_splits * (unsigned long long)(d + 1) * sizeof(float);
    if (need > FLASHD_STATIC_SCRATCH_BYTES) return FLASHD_ERR_WORKSPACE;   // beyond the fixed scratch
    float* ws = static_scratch_ptr();
    if (ws == nullptr) return FLASHD_ERR_CUDA;
    cudaStream_t s = as_stream(stream);
    const int ps = (d == 128) ? launch_partial<128>(q, k, v, ws, rows, Nq, Nk, scale, num_splits, s)
                              : launch_partial<64>(q, k, v, ws, rows, Nq, Nk, scale, num_splits, s);
    if (ps != FLASHD_OK) return ps;
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(o);
    if (d == 128) splitk_combine_kernel<128, __nv_bfloat16><<<(unsigned)rows, 128, 0, s>>>(ws, out, nullptr, num_splits);
    else splitk_combine_kernel<64, __nv_bfloat16><<<(unsigned)rows, 64, 0, s>>>(ws, out, nullptr, num_splits);
    return after_launch();
}

int flashd_skip_stats(const void* q, const void* k, unsigned long long* counts, int in_dtype, int B, int H, int Nq,
                      int Nk, int d, float scale, int causal, float lo, float hi, float alo, float ahi,
                      void* stream) {
    if (!q || !k || !counts) return FLASHD_ERR_NULL;
    if (B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0 || d <= 0 || !std::isfinite(scale)) return FLASHD_ERR_SHAPE;
    if (!(lo <= hi) || !(alo <= ahi)) return FLASHD_ERR_SHAPE;
    if (!aligned16(q) || !aligned16(k) || (reinterpret_cast<uintptr_t>(counts) & 7u)) return FLASHD_ERR_ALIGN;
    if (d != 16 && d != 32 && d != 64 && d != 128 && d != 256) return FLASHD_ERR_UNSUPPORTED;
    if (in_dtype != FLASHD_BF16 && in_dtype != FLASHD_F32) return FLASHD_ERR_UNSUPPORTED;
    const long long rows = (long long)B * H * Nq;
    const int warps = 4;
    const long long blocks = (rows + warps - 1) / warps;
    if (blocks > 0x7fffffffLL) return FLASHD_ERR_SHAPE;
    cudaStream_t s = as_stream(stream);
    if (cudaMemsetAsync(counts, 0, 5 * sizeof(unsigned long long), s) != cudaSuccess) return FLASHD_ERR_CUDA;
#define FLASHD_LAUNCH_STATS(T, E) \
    skipstats_kernel<T, E><<<(unsigned)blocks, warps * 32, 0, s>>>(static_cast<const T*>(q), static_cast<const T*>(k), \
                                                                  counts, rows, Nq, Nk, scale, causal, lo, hi, alo, ahi)
    if (in_dtype == FLASHD_BF16) {
        switch (d) {
            case 32: FLASHD_LAUNCH_STATS(__nv_bfloat16, 1); break;
            case 64: FLASHD_LAUNCH_STATS(__nv_bfloat16, 2); break;
            case 128: FLASHD_LAUNCH_STATS(__nv_bfloat16, 4); break;
            default: FLASHD_LAUNCH_STATS(__nv_bfloat16, 8); break;
        }
    } else {
        switch (d) {
            case 32: FLASHD_LAUNCH_STATS(float, 1); break;
            case 64: FLASHD_LAUNCH_STATS(float, 2); break;
            case 128: FLASHD_LAUNCH_STATS(float, 4); break;
            default: FLASHD_LAUNCH_STATS(float, 8); break;
        }
    }
#undef FLASHD_LAUNCH_STATS
    return after_launch();
}

int flashd_attn_fwd_host(const void* q, const void* k, const void* v, void* o, int path, int B, int H, int Nq,
                         int Nk, int d, float scale, int causal, void* stream) {
    if (!q || !k || !v || !o) return FLASHD_ERR_NULL;
    if (B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0 || d <= 0 || !std::isfinite(scale)) return FLASHD_ERR_SHAPE;
    if (path < 0 || path > 2) return FLASHD_ERR_UNSUPPORTED;
    if (path == 2 && causal) return FLASHD_ERR_UNSUPPORTED;
    if ((long long)B * H > 0x7fffffffLL / 2) return FLASHD_ERR_SHAPE;
    const size_t esz = (path == 1) ? 4 : 2;
    const int BH = B * H;
    const size_t q_head = (size_t)Nq * d * esz, k_head = (size_t)Nk * d * esz;   // bytes of one head
    const size_t qb = q_head * BH, kb = k_head * BH;
    cudaStream_t s = as_stream(stream);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FLASHD_ERR_CUDA;
    // keep freed staging buffers in the device's default pool instead of returning them to
    // the driver at every synchronisation (set once per device)
    {
        static bool pool_set[64] = {false};
        if (!pool_set[dev]) {
            cudaMemPool_t pool;
            if (cudaDeviceGetDefaultMemPool(&pool, dev) == cudaSuccess) {
                unsigned long long keep = ~0ull;
                cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
            }
            pool_set[dev] = true;
        }
    }
    // Heads are independent, so the batch is cut into chunks of whole heads and the three
    // legs are pipelined on three streams: chunk c+1 is copied in while chunk c is computed
    // and chunk c-1 is copied out (the two copy directions use different copy engines).
    // About 12 MB of input per chunk, at most 8 chunks: every chunk costs some tens of
    // microseconds of copy set-up, so finer cuts lose more than they overlap.
    int chunks = (int)std::min<size_t>(8, std::max<size_t>(1, (qb + 2 * kb) / (12u << 20)));
    if (chunks > BH) chunks = BH;
    const int heads_per = (BH + chunks - 1) / chunks;
    chunks = (BH + heads_per - 1) / heads_per;
    int splits = 0;
    size_t wsb = 0;
    if (path == 2) {
        splits = flashd_splitk_num_splits(1, heads_per, Nq, Nk, d);
        wsb = flashd_splitk_workspace_bytes(1, heads_per, Nq, d, splits);
    }
    std::lock_guard<std::mutex> lock(g_pipe_mutex);     // the helper streams and events are shared per device
    HostPipe& hp = g_pipe[dev];
    if (!host_pipe_init(hp)) return FLASHD_ERR_CUDA;
    char *dq = nullptr, *dk = nullptr, *dv = nullptr, *dout = nullptr;
    void* dws = nullptr;
    int st = FLASHD_OK;
    bool ok = cudaMallocAsync((void**)&dq, qb, s) == cudaSuccess && cudaMallocAsync((void**)&dk, kb, s) == cudaSuccess &&
              cudaMallocAsync((void**)&dv, kb, s) == cudaSuccess && cudaMallocAsync((void**)&dout, qb, s) == cudaSuccess &&
              (wsb == 0 || cudaMallocAsync(&dws, wsb, s) == cudaSuccess);
    // the helper streams start after everything already queued on `stream` (and the allocations)
    ok = ok && cudaEventRecord(hp.ev_start, s) == cudaSuccess &&
         cudaStreamWaitEvent(hp.s_in, hp.ev_start, 0) == cudaSuccess &&
         cudaStreamWaitEvent(hp.s_out, hp.ev_start, 0) == cudaSuccess;
    if (!ok) st = FLASHD_ERR_CUDA;
    for (int c = 0; c < chunks && st == FLASHD_OK; ++c) {
        const int h0 = c * heads_per;
        const int nh = std::min(heads_per, BH - h0);
        const size_t qo = q_head * h0, ko = k_head * h0;
        ok = cudaMemcpyAsync(dq + qo, static_cast<const char*>(q) + qo, q_head * nh, cudaMemcpyHostToDevice, hp.s_in) == cudaSuccess &&
             cudaMemcpyAsync(dk + ko, static_cast<const char*>(k) + ko, k_head * nh, cudaMemcpyHostToDevice, hp.s_in) == cudaSuccess &&
             cudaMemcpyAsync(dv + ko, static_cast<const char*>(v) + ko, k_head * nh, cudaMemcpyHostToDevice, hp.s_in) == cudaSuccess &&
             cudaEventRecord(hp.ev_in[c], hp.s_in) == cudaSuccess && cudaStreamWaitEvent(s, hp.ev_in[c], 0) == cudaSuccess;
        if (!ok) { st = FLASHD_ERR_CUDA; break; }
        if (path == 0) st = flashd_attn_fwd(dq + qo, dk + ko, dv + ko, dout + qo, 1, nh, Nq, Nk, d, scale, causal, stream);
        else if (path == 1) st = flashd_attn_fwd_f32(dq + qo, dk + ko, dv + ko, dout + qo, 1, nh, Nq, Nk, d, scale, causal, stream);
        else st = flashd_attn_fwd_splitk(dq + qo, dk + ko, dv + ko, dout + qo, dws, wsb, 1, nh, Nq, Nk, d, scale,
                                         nh == heads_per ? splits : 0, stream);
        if (st != FLASHD_OK) break;
        ok = cudaEventRecord(hp.ev_k[c], s) == cudaSuccess && cudaStreamWaitEvent(hp.s_out, hp.ev_k[c], 0) == cudaSuccess &&
             cudaMemcpyAsync(static_cast<char*>(o) + qo, dout + qo, q_head * nh, cudaMemcpyDeviceToHost, hp.s_out) == cudaSuccess;
        if (!ok) st = FLASHD_ERR_CUDA;
    }
    // `stream` rejoins the helper streams before the buffers go back to the pool
    if (cudaEventRecord(hp.ev_out, hp.s_out) != cudaSuccess || cudaStreamWaitEvent(s, hp.ev_out, 0) != cudaSuccess ||
        cudaEventRecord(hp.ev_start, hp.s_in) != cudaSuccess || cudaStreamWaitEvent(s, hp.ev_start, 0) != cudaSuccess) {
        if (st == FLASHD_OK) st = FLASHD_ERR_CUDA;
        cudaStreamSynchronize(hp.s_in);
        cudaStreamSynchronize(hp.s_out);
    }
    if (dq) cudaFreeAsync(dq, s);
    if (dk) cudaFreeAsync(dk, s);
    if (dv) cudaFreeAsync(dv, s);
    if (dout) cudaFreeAsync(dout, s);
    if (dws) cudaFreeAsync(dws, s);
    if (cudaStreamSynchronize(s) != cudaSuccess && st == FLASHD_OK) st = FLASHD_ERR_CUDA;
    return st;
}

int flashd_last_device_status(void* stream, int* detail) {
    if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) return FLASHD_ERR_CUDA;
    unsigned int h[4] = {0, 0, 0, 0};
    if (cudaMemcpyFromSymbol(h, flashd::g_status, sizeof(h)) != cudaSuccess) return FLASHD_ERR_CUDA;
    if (h[0] != 0) {
        const unsigned int z[4] = {0, 0, 0, 0};
        cudaMemcpyToSymbol(flashd::g_status, z, sizeof(z));
    }
    if (detail) for (int i = 0; i < 4; ++i) detail[i] = (int)h[i];
    return (int)h[0];
}

}  // extern "C"
