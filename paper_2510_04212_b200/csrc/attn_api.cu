// C ABI of the library (see include/attn.h): argument validation, TMA descriptor
// construction and kernel launches.  No device memory is allocated here; the only
// device-resident state is a status word in static device memory.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <atomic>
#include <utility>

#include "../../include/attn.h"
#include "bwd_kernel.cuh"
#include "bwd_kernel_d64.cuh"
#include "packed_copy_kernel.cuh"
#include "quantize_v_kernel.cuh"
#include "bwd_kernel_d128.cuh"
#include "delta_dp_kernel.cuh"
#include "fwd_kernel.cuh"
#include "selftest_kernel.cuh"

// Scratch for attn_bwd_static(): lives in the library's device image, so every GPU that loads the
// library holds these bytes until the process exits.  In host code this name is only a handle for
// cudaGetSymbolAddress(); it is not a device address and must never be passed to a kernel as one.
static __device__ __align__(256) unsigned char g_static_bwd_scratch[ATTN_BWD_STATIC_MAX_BYTES];

namespace {

__device__ int g_device_status = 0;       // set by a kernel: 1 = a bounded wait ran out, 2 = shared-memory layout check failed

// Host-side state.  Entry points may be called from several host threads at once (each with its own current device
// and stream): the process-wide parameters are atomics, everything cached per device is an array indexed by the
// device ordinal and written once with release / read with acquire.
constexpr int MAX_DEVICES = 64;
std::atomic<float> g_beta{2.0f};
std::atomic<float> g_eps{1e-3f};
std::atomic<float> g_guard_cap{ATTN_GUARD_DEFAULT_MAX_SHIFT};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encoder()
{
    static std::atomic<EncodeTiledFn> fn{nullptr};
    EncodeTiledFn f = fn.load(std::memory_order_acquire);
    if (!f) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        f = reinterpret_cast<EncodeTiledFn>(p);
        fn.store(f, std::memory_order_release);     // two threads may both look it up: they store the same pointer
    }
    return f;
}

// [rows, d] BF16 row-major viewed as a 2D tensor; one box = box_rows rows x 64 columns (128 bytes,
// the span of the 128-byte shared-memory swizzle).
bool make_map(CUtensorMap* m, const void* base, long long rows, int d, int box_rows = 128)
{
    EncodeTiledFn enc = get_encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(d) * 2};
    const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// V transposed, one-byte elements: [rows = B*H*d][N keys]; one box = d rows x 64 keys (64 bytes), 64-byte swizzle.
bool make_map_vt_u8(CUtensorMap* m, const void* base, long long rows, int N, int d)
{
    EncodeTiledFn enc = get_encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(N)};
    const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(d)};
    const cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [rows, d] FP32 row-major; one box = 128 rows x 32 columns (128 bytes).
bool make_map_f32(CUtensorMap* m, const void* base, long long rows, int d)
{
    EncodeTiledFn enc = get_encoder();
    if (!enc) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(d) * 4};
    const cuuint32_t box[2] = {32, 128};
    const cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int check_shape(int B, int H, int N, int d)
{
    if (B < 1 || H < 1 || N < 128 || (N % 128) != 0) return ATTN_ERR_SHAPE;
    if (d != 64 && d != 128) return ATTN_ERR_SHAPE;
    if (static_cast<long long>(B) * H * N >= (1ll << 31)) return ATTN_ERR_SHAPE;
    return ATTN_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Compute-capability major and SM count of the current device, looked up once per device.
struct DeviceInfo { int major, sm_count; };
int device_info(DeviceInfo* out, int* dev_out = nullptr)
{
    static std::atomic<int> packed[MAX_DEVICES];      // 0 = not looked up yet; else (major << 16) | sm_count
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return ATTN_ERR_CUDA;
    int v = packed[dev].load(std::memory_order_acquire);
    if (!v) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || major <= 0 || sms <= 0)
            return ATTN_ERR_CUDA;
        v = (major << 16) | sms;
        packed[dev].store(v, std::memory_order_release);
    }
    out->major = v >> 16;
    out->sm_count = v & 0xFFFF;
    if (dev_out) *dev_out = dev;
    return ATTN_OK;
}

int check_device()
{
    DeviceInfo di;
    if (int e = device_info(&di)) return e;
    return di.major == 10 ? ATTN_OK : ATTN_ERR_DEVICE;
}

// cudaFuncAttributeMaxDynamicSharedMemorySize is per device and per kernel: set it once for each (kernel, device).
template <auto Kern>
int ensure_dynamic_smem(int bytes)
{
    static std::atomic<bool> done[MAX_DEVICES];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return ATTN_ERR_CUDA;
    if (!done[dev].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(Kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return ATTN_ERR_CUDA;
        done[dev].store(true, std::memory_order_release);
    }
    return ATTN_OK;
}

int* status_ptr()
{
    int* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_device_status) != cudaSuccess) return nullptr;
    return p;
}

// Every kernel of the library is launched with programmatic stream serialization: its CTAs may be scheduled while
// the kernel before it in the stream is draining, set up their barriers and TMEM, and then wait (griddepcontrol.wait)
// for that kernel to complete before they touch global memory.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

template <int D, int MODE, bool CAUSAL, bool COUNT, bool PADDED = false, bool FP8PV = false>
int launch_fwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
               const attn::FwdParams& prm, cudaStream_t st)
{
    using Cfg = attn::FwdCfg<D>;
    constexpr auto kern = attn::attn_fwd_kernel<D, MODE, CAUSAL, COUNT, PADDED, FP8PV>;
    if (int e = ensure_dynamic_smem<kern>(Cfg::SMEM_BYTES)) return e;
    return launch_pdl(kern, dim3(prm.Tr * prm.BH), dim3(Cfg::THREADS), Cfg::SMEM_BYTES, st, tq, tk, tv, to, prm) == cudaSuccess
               ? ATTN_OK : ATTN_ERR_CUDA;
}

template <bool CAUSAL, bool GENERAL>
int launch_bwd_d128(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                    const CUtensorMap& tdk, const CUtensorMap& tdv, const attn::BwdParams& prm, cudaStream_t st)
{
    using Cfg = attn::Bwd128Cfg;
    constexpr auto kern = attn::attn_bwd_kernel_d128<CAUSAL, GENERAL>;
    if (int e = ensure_dynamic_smem<kern>(Cfg::SMEM_BYTES)) return e;
    return launch_pdl(kern, dim3(prm.Tr * prm.BH), dim3(Cfg::THREADS), Cfg::SMEM_BYTES, st, tq, tk, tv, tdo, tdk, tdv,
                      prm) == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

template <bool CAUSAL, bool GENERAL>
int launch_bwd_d64(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                   const CUtensorMap& tdk, const CUtensorMap& tdv, const CUtensorMap& tacc,
                   const attn::BwdParams& prm, cudaStream_t st)
{
    using Cfg = attn::Bwd64Cfg;
    constexpr auto kern = attn::attn_bwd_kernel_d64<CAUSAL, GENERAL>;
    if (int e = ensure_dynamic_smem<kern>(Cfg::SMEM_BYTES)) return e;
    DeviceInfo di;
    if (int e = device_info(&di)) return e;
    const int sm_count = di.sm_count;
    // persistent: one CTA per SM walks the (head, key tile) items
    const long long items = static_cast<long long>(prm.Tr) * prm.BH;
    const unsigned grid = static_cast<unsigned>(items < sm_count ? items : sm_count);
    if (launch_pdl(kern, dim3(grid), dim3(Cfg::THREADS), Cfg::SMEM_BYTES, st, tq, tk, tv, tdo, tdk, tdv, tacc, prm) != cudaSuccess)
        return ATTN_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

// delta != nullptr: computed and stored; delta_given != nullptr: taken from the caller; lse, dq_acc, dq_tiles: only for
// the full backward (nullptr for the stand-alone delta pass)
int launch_preprocess(const void* o, const void* dO, float* delta, const float* delta_given, const float* lse,
                      float* dq_acc, void* dq_tiles, long long rows, int d, cudaStream_t st)
{
    const long long n_chunks = rows * (d / 8);
    const int threads = 256;
    const long long blocks = (n_chunks + threads - 1) / threads;
    cudaError_t e;
    if (d == 64)
        e = launch_pdl(attn::bwd_preprocess_kernel<64>, dim3(static_cast<unsigned>(blocks)), dim3(threads), 0, st,
                       static_cast<const uint4*>(o), static_cast<const uint4*>(dO), delta, delta_given, lse,
                       reinterpret_cast<float4*>(dq_acc), static_cast<uint8_t*>(dq_tiles), n_chunks);
    else
        e = launch_pdl(attn::bwd_preprocess_kernel<128>, dim3(static_cast<unsigned>(blocks)), dim3(threads), 0, st,
                       static_cast<const uint4*>(o), static_cast<const uint4*>(dO), delta, delta_given, lse,
                       reinterpret_cast<float4*>(dq_acc), static_cast<uint8_t*>(dq_tiles), n_chunks);
    return e == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

template <int D, bool CAUSAL>
int launch_delta_dp(const void* q, const void* k, const void* v, const void* dO, const float* lse, float* delta,
                           int BH, int N, float scale, cudaStream_t st)
{
    using Cfg = attn::DeltaDpCfg<D>;
    constexpr auto kern = attn::delta_dp_kernel<D, CAUSAL>;
    if (int e = ensure_dynamic_smem<kern>(Cfg::SMEM_BYTES)) return e;
    kern<<<static_cast<unsigned>((N / Cfg::ROWS) * BH), 256, Cfg::SMEM_BYTES, st>>>(
        static_cast<const uint4*>(q), static_cast<const uint4*>(k), static_cast<const uint4*>(v),
        static_cast<const uint4*>(dO), lse, delta, N, scale);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

}  // namespace

extern "C" {

// attn_fwd and attn_fwd_count_ones: `ones` == nullptr selects the instantiations without the counter
static int fwd_impl(const void* q, const void* k, const void* v, void* o, float* lse, int* ones,
                    int B, int H, int Hkv, int N, int seqlen, const int* seqlens, int d, int causal, float scale, int mode,
                    void* stream, int pbar_fmt = ATTN_PBAR_BF16, float* o_f32 = nullptr, float fp8_v_descale = 0.0f)
{
    const bool fp8pv = fp8_v_descale != 0.0f;       // v is then V^T in E4M3, [B][H][d][N]
    if (pbar_fmt != ATTN_PBAR_BF16 && pbar_fmt != ATTN_PBAR_E4M3 && pbar_fmt != ATTN_PBAR_E5M2) return ATTN_ERR_MODE;
    if (!q || !k || !v || !o || !lse) return ATTN_ERR_NULL;
    if (int e = check_shape(B, H, N, d)) return e;
    if (Hkv < 1 || H % Hkv != 0) return ATTN_ERR_SHAPE;
    if (seqlen < 1 || seqlen > N) return ATTN_ERR_SHAPE;
    if (mode & ~(ATTN_MODE_STABILISED | ATTN_MODE_FLAG_SINGLE_ROUNDING | ATTN_MODE_FLAG_GUARDED)) return ATTN_ERR_MODE;
    if ((mode & ATTN_MODE_FLAG_GUARDED) && !(mode & ATTN_MODE_STABILISED)) return ATTN_ERR_MODE;
    if (!(scale > 0.0f) || !isfinite(scale)) return ATTN_ERR_PARAM;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return ATTN_ERR_ALIGN;
    if (int e = check_device()) return e;
    int* status = status_ptr();
    if (!status) return ATTN_ERR_CUDA;

    const long long rows = static_cast<long long>(B) * H * N;
    CUtensorMap tq, tk, tv, to;
    const int bc = attn::FwdCfg<64>::BC;
    const long long kvrows = static_cast<long long>(B) * Hkv * N;
    if (!make_map(&tq, q, rows, d, 128) || !make_map(&tk, k, kvrows, d, bc) || !make_map(&to, o, rows, d, 128))
        return ATTN_ERR_CUDA;
    if (!(fp8pv ? make_map_vt_u8(&tv, v, static_cast<long long>(B) * Hkv * d, N, d) : make_map(&tv, v, kvrows, d, bc)))
        return ATTN_ERR_CUDA;

    attn::FwdParams prm;
    prm.lse = lse;
    prm.ones = ones;
    prm.o_f32 = o_f32;
    prm.pbar_fmt = pbar_fmt;
    prm.single_rounding = (mode & ATTN_MODE_FLAG_SINGLE_ROUNDING) ? 1 : 0;
    prm.N = N;
    prm.BH = B * H;
    prm.Tr = (seqlen + 127) / 128;
    prm.seqlen = seqlen;
    prm.seqlens = seqlens;
    prm.H = H;
    prm.group = H / Hkv;
    prm.scale = scale;
    prm.beta = g_beta.load();
    prm.eps = g_eps.load();
    prm.guard_cap = (mode & ATTN_MODE_FLAG_GUARDED) ? g_guard_cap.load() : 0.0f;
    prm.v_descale = fp8_v_descale;
    prm.status = status;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (fp8pv) {
        const bool m1 = (mode & ATTN_MODE_STABILISED) != 0;
        if (d == 64) {
            if (causal) return m1 ? launch_fwd<64, 1, true, false, false, true>(tq, tk, tv, to, prm, st)
                                  : launch_fwd<64, 0, true, false, false, true>(tq, tk, tv, to, prm, st);
            return m1 ? launch_fwd<64, 1, false, false, false, true>(tq, tk, tv, to, prm, st)
                      : launch_fwd<64, 0, false, false, false, true>(tq, tk, tv, to, prm, st);
        }
        if (causal) return m1 ? launch_fwd<128, 1, true, false, false, true>(tq, tk, tv, to, prm, st)
                              : launch_fwd<128, 0, true, false, false, true>(tq, tk, tv, to, prm, st);
        return m1 ? launch_fwd<128, 1, false, false, false, true>(tq, tk, tv, to, prm, st)
                  : launch_fwd<128, 0, false, false, false, true>(tq, tk, tv, to, prm, st);
    }
    const int key = (d == 128 ? 8 : 0) | ((mode & ATTN_MODE_STABILISED) ? 4 : 0) | (causal ? 2 : 0) | ((ones || o_f32) ? 1 : 0);
    // full attention over a sequence that ends inside a 64-key tile: the instantiations that mask the rest of that tile
    if (!causal && (seqlen % bc != 0 || seqlens)) {
        if (ones || o_f32) return ATTN_ERR_SHAPE;
        const bool m1 = (mode & ATTN_MODE_STABILISED) != 0;
        if (d == 64) return m1 ? launch_fwd<64, 1, false, false, true>(tq, tk, tv, to, prm, st)
                               : launch_fwd<64, 0, false, false, true>(tq, tk, tv, to, prm, st);
        return m1 ? launch_fwd<128, 1, false, false, true>(tq, tk, tv, to, prm, st)
                  : launch_fwd<128, 0, false, false, true>(tq, tk, tv, to, prm, st);
    }
    switch (key) {
#define FWD_CASE(K, D_, M_, C_, N_) case K: return launch_fwd<D_, M_, C_, N_>(tq, tk, tv, to, prm, st);
        FWD_CASE(0, 64, 0, false, false)   FWD_CASE(1, 64, 0, false, true)
        FWD_CASE(2, 64, 0, true, false)    FWD_CASE(3, 64, 0, true, true)
        FWD_CASE(4, 64, 1, false, false)   FWD_CASE(5, 64, 1, false, true)
        FWD_CASE(6, 64, 1, true, false)    FWD_CASE(7, 64, 1, true, true)
        FWD_CASE(8, 128, 0, false, false)  FWD_CASE(9, 128, 0, false, true)
        FWD_CASE(10, 128, 0, true, false)  FWD_CASE(11, 128, 0, true, true)
        FWD_CASE(12, 128, 1, false, false) FWD_CASE(13, 128, 1, false, true)
        FWD_CASE(14, 128, 1, true, false)  FWD_CASE(15, 128, 1, true, true)
#undef FWD_CASE
    }
    return ATTN_ERR_PARAM;
}

int attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
             int B, int H, int N, int d, int causal, float scale, int mode, void* stream)
{
    return fwd_impl(q, k, v, o, lse, nullptr, B, H, H, N, N, nullptr, d, causal, scale, mode, stream);
}

int attn_fwd_count_ones(const void* q, const void* k, const void* v, void* o, float* lse, int* ones,
                        int B, int H, int N, int d, int causal, float scale, int mode, void* stream)
{
    if (!ones) return ATTN_ERR_NULL;
    return fwd_impl(q, k, v, o, lse, ones, B, H, H, N, N, nullptr, d, causal, scale, mode, stream);
}

int attn_fwd_pbar_format(const void* q, const void* k, const void* v, void* o, float* lse, int* ones,
                         int B, int H, int N, int d, int causal, float scale, int mode, int pbar_format, void* stream)
{
    if (!ones) return ATTN_ERR_NULL;
    return fwd_impl(q, k, v, o, lse, ones, B, H, H, N, N, nullptr, d, causal, scale, mode, stream, pbar_format);
}

int attn_quantize_v_e4m3(const void* v, void* v_t_e4m3, int B, int H, int N, int d, float v_scale, void* stream)
{
    if (!v || !v_t_e4m3) return ATTN_ERR_NULL;
    if (int e = check_shape(B, H, N, d)) return e;
    if (!(v_scale > 0.0f) || !isfinite(v_scale)) return ATTN_ERR_PARAM;
    if (!aligned16(v) || !aligned16(v_t_e4m3)) return ATTN_ERR_ALIGN;
    if (int e = check_device()) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const dim3 grid(static_cast<unsigned>(N / (16 * (256 / d))), static_cast<unsigned>(B * H));
    if (d == 64)
        attn::quantize_v_e4m3_kernel<64><<<grid, 256, 0, st>>>(static_cast<const uint16_t*>(v), static_cast<uint8_t*>(v_t_e4m3), N, v_scale);
    else
        attn::quantize_v_e4m3_kernel<128><<<grid, 256, 0, st>>>(static_cast<const uint16_t*>(v), static_cast<uint8_t*>(v_t_e4m3), N, v_scale);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

int attn_fwd_fp8pv(const void* q, const void* k, const void* v_t_e4m3, void* o, float* lse,
                   int B, int H, int N, int d, int causal, float scale, int mode, float v_descale, void* stream)
{
    if (!(v_descale > 0.0f) || !isfinite(v_descale)) return ATTN_ERR_PARAM;
    if (mode & ~ATTN_MODE_STABILISED) return ATTN_ERR_MODE;
    return fwd_impl(q, k, v_t_e4m3, o, lse, nullptr, B, H, H, N, N, nullptr, d, causal, scale, mode, stream, ATTN_PBAR_BF16,
                    nullptr, v_descale);
}

int attn_fwd_o_f32(const void* q, const void* k, const void* v, void* o, float* lse, float* o_f32,
                   int B, int H, int N, int d, int causal, float scale, int mode, void* stream)
{
    if (!o_f32) return ATTN_ERR_NULL;
    if (!aligned16(o_f32)) return ATTN_ERR_ALIGN;
    return fwd_impl(q, k, v, o, lse, nullptr, B, H, H, N, N, nullptr, d, causal, scale, mode, stream, ATTN_PBAR_BF16, o_f32);
}

int attn_bwd_delta_f32(const float* o_f32, const void* dO, float* delta, int B, int H, int N, int d, void* stream)
{
    if (!o_f32 || !dO || !delta) return ATTN_ERR_NULL;
    if (int e = check_shape(B, H, N, d)) return e;
    if (!aligned16(o_f32) || !aligned16(dO)) return ATTN_ERR_ALIGN;
    if (int e = check_device()) return e;
    const long long n_chunks = static_cast<long long>(B) * H * N * (d / 8);
    const unsigned blocks = static_cast<unsigned>((n_chunks + 255) / 256);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (d == 64)
        attn::delta_f32_kernel<64><<<blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(o_f32), static_cast<const uint4*>(dO), delta, n_chunks);
    else
        attn::delta_f32_kernel<128><<<blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(o_f32), static_cast<const uint4*>(dO), delta, n_chunks);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

int attn_bwd_preprocess(const void* o, const void* dO, float* delta, int B, int H, int N, int d, void* stream)
{
    if (!o || !dO || !delta) return ATTN_ERR_NULL;
    if (int e = check_shape(B, H, N, d)) return e;
    if (!aligned16(o) || !aligned16(dO)) return ATTN_ERR_ALIGN;
    if (int e = check_device()) return e;
    return launch_preprocess(o, dO, delta, nullptr, nullptr, nullptr, nullptr, static_cast<long long>(B) * H * N, d,
                             static_cast<cudaStream_t>(stream));
}

int attn_bwd_delta_dp(const void* q, const void* k, const void* v, const void* dO, const float* lse, float* delta,
                      int B, int H, int N, int d, int causal, float scale, void* stream)
{
    if (!q || !k || !v || !dO || !lse || !delta) return ATTN_ERR_NULL;
    if (int e = check_shape(B, H, N, d)) return e;
    if (!(scale > 0.0f) || !isfinite(scale)) return ATTN_ERR_PARAM;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(dO)) return ATTN_ERR_ALIGN;
    if (int e = check_device()) return e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int BH = B * H;
    if (d == 64) return causal ? launch_delta_dp<64, true>(q, k, v, dO, lse, delta, BH, N, scale, st)
                               : launch_delta_dp<64, false>(q, k, v, dO, lse, delta, BH, N, scale, st);
    return causal ? launch_delta_dp<128, true>(q, k, v, dO, lse, delta, BH, N, scale, st)
                  : launch_delta_dp<128, false>(q, k, v, dO, lse, delta, BH, N, scale, st);
}

size_t attn_bwd_workspace_bytes(int B, int H, int N, int d)
{
    if (check_shape(B, H, N, d) != ATTN_OK) return 0;
    return static_cast<size_t>(B) * H * N * d * sizeof(float);
}

static int bwd_stage_impl(int stage, const void* q, const void* k, const void* v, const void* o, const void* dO,
                          const float* lse, void* dq, void* dk, void* dv, float* delta, void* workspace,
                          size_t workspace_bytes, int B, int H, int Hkv, int N, int seqlen, const int* seqlens, int d,
                          int causal, float scale, int mode, void* stream)
{
    if (stage < ATTN_BWD_STAGE_ALL || stage > ATTN_BWD_STAGE_FINALIZE) return ATTN_ERR_PARAM;
    if (!q || !k || !v || !o || !dO || !lse || !dq || !dk || !dv || !delta) return ATTN_ERR_NULL;
    if (int e = check_shape(B, H, N, d)) return e;
    if (Hkv < 1 || H % Hkv != 0) return ATTN_ERR_SHAPE;
    if (seqlen < 1 || seqlen > N) return ATTN_ERR_SHAPE;
    if (mode & ~(ATTN_MODE_STABILISED | ATTN_MODE_FLAG_SINGLE_ROUNDING | ATTN_MODE_FLAG_DELTA_GIVEN)) return ATTN_ERR_MODE;
    if (!(scale > 0.0f) || !isfinite(scale)) return ATTN_ERR_PARAM;
    if (!workspace || workspace_bytes < attn_bwd_workspace_bytes(B, H, N, d) ||
        (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
        return ATTN_ERR_WORKSPACE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(dO) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv))
        return ATTN_ERR_ALIGN;
    if (int e = check_device()) return e;
    int* status = status_ptr();
    if (!status) return ATTN_ERR_CUDA;

    const long long rows = static_cast<long long>(B) * H * N;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* acc = static_cast<float*>(workspace);
    const bool all = stage == ATTN_BWD_STAGE_ALL;

    // 1. delta = rowsum(dO o O); the same pass clears the dQ accumulator and writes, into the bytes of every 128-row
    //    tile of the dQ output buffer, the tile's arrival counter and its per-query vectors for the main kernel
    if (all || stage == ATTN_BWD_STAGE_PREPROCESS) {
        const bool given = (mode & ATTN_MODE_FLAG_DELTA_GIVEN) != 0;
        if (int e = launch_preprocess(o, dO, given ? nullptr : delta, given ? delta : nullptr, lse, acc, dq, rows, d, st))
            return e;
    }

    // 2. dK, dV and the FP32 dQ accumulator
    if (all || stage == ATTN_BWD_STAGE_MAIN) {
        CUtensorMap tq, tk, tv, tdo;
        const long long kvrows = static_cast<long long>(B) * Hkv * N;      // K, V, dK, dV: [B][Hkv][N][d]
        if (!make_map(&tq, q, rows, d) || !make_map(&tk, k, kvrows, d) || !make_map(&tv, v, kvrows, d) ||
            !make_map(&tdo, dO, rows, d))
            return ATTN_ERR_CUDA;
        attn::BwdParams prm;
        prm.lse = lse;
        prm.delta = delta;
        prm.dq_acc = acc;
        prm.dq = static_cast<uint16_t*>(dq);
        prm.dk = static_cast<uint16_t*>(dk);
        prm.dv = static_cast<uint16_t*>(dv);
        prm.N = N;
        prm.BH = B * Hkv;
        prm.Tr = (seqlen + 127) / 128;
        prm.seqlen = seqlen;
        prm.seqlens = seqlens;
        prm.Hkv = Hkv;
        prm.group = H / Hkv;
        {   // Heads in flight together in the causal d = 128 kernel: about 64 MB of Q, dO, K, V and FP32 dQ accumulator,
            // a divisor of the head count (a smaller last group would start its long key tiles last: measured slower
            // than no grouping), and enough of them to give every SM a CTA one and a half times over.
            const long long per_head = static_cast<long long>(N) * d * (prm.group * 8 + 4);
            const long long target = (64ll << 20) / per_head;
            int hg = 1;
            for (int c = 1; c <= prm.BH; ++c)
                if (prm.BH % c == 0 && (c <= target || static_cast<long long>(hg) * prm.Tr < 222)) hg = c; else if (prm.BH % c == 0) break;
            prm.head_group = hg;
        }
        prm.scale = scale;
        prm.status = status;
        int e;
        if (d == 64) {
            CUtensorMap tdk, tdv, tacc;
            if (!make_map(&tdk, dk, kvrows, d) || !make_map(&tdv, dv, kvrows, d) || !make_map_f32(&tacc, acc, rows, d))
                return ATTN_ERR_CUDA;
            if (prm.group == 1 && seqlen % 128 == 0 && !seqlens)      // the plain instantiation: no group arithmetic, only the diagonal masked
                e = causal ? launch_bwd_d64<true, false>(tq, tk, tv, tdo, tdk, tdv, tacc, prm, st)
                           : launch_bwd_d64<false, false>(tq, tk, tv, tdo, tdk, tdv, tacc, prm, st);
            else
                e = causal ? launch_bwd_d64<true, true>(tq, tk, tv, tdo, tdk, tdv, tacc, prm, st)
                           : launch_bwd_d64<false, true>(tq, tk, tv, tdo, tdk, tdv, tacc, prm, st);
        } else {
            CUtensorMap tdk, tdv;
            if (!make_map(&tdk, dk, kvrows, d) || !make_map(&tdv, dv, kvrows, d)) return ATTN_ERR_CUDA;
            if (prm.group == 1 && seqlen % 128 == 0 && !seqlens)
                e = causal ? launch_bwd_d128<true, false>(tq, tk, tv, tdo, tdk, tdv, prm, st)
                           : launch_bwd_d128<false, false>(tq, tk, tv, tdo, tdk, tdv, prm, st);
            else
                e = causal ? launch_bwd_d128<true, true>(tq, tk, tv, tdo, tdk, tdv, prm, st)
                           : launch_bwd_d128<false, true>(tq, tk, tv, tdo, tdk, tdv, prm, st);
        }
        if (e) return e;
    }

    // 3. dQ = bf16(scale * accumulator); for d = 64 the main kernel has already done this tile by tile
    if ((all || stage == ATTN_BWD_STAGE_FINALIZE) && d != 64) {
        const long long n_chunks = rows * (d / 8);
        const int threads = 256;
        if (launch_pdl(attn::dq_convert_tiled128_kernel, dim3(static_cast<unsigned>((n_chunks + threads - 1) / threads)),
                       dim3(threads), 0, st, reinterpret_cast<const float4*>(acc), static_cast<uint4*>(dq), scale,
                       n_chunks) != cudaSuccess)
            return ATTN_ERR_CUDA;
    }
    return ATTN_OK;
}

int attn_bwd_stage(int stage, const void* q, const void* k, const void* v, const void* o, const void* dO,
                   const float* lse, void* dq, void* dk, void* dv, float* delta, void* workspace,
                   size_t workspace_bytes, int B, int H, int N, int d, int causal, float scale, int mode,
                   void* stream)
{
    return bwd_stage_impl(stage, q, k, v, o, dO, lse, dq, dk, dv, delta, workspace, workspace_bytes, B, H, H, N, N,
                          nullptr, d, causal, scale, mode, stream);
}

int attn_fwd_gqa(const void* q, const void* k, const void* v, void* o, float* lse,
                 int B, int H, int H_kv, int N, int d, int causal, float scale, int mode, void* stream)
{
    return fwd_impl(q, k, v, o, lse, nullptr, B, H, H_kv, N, N, nullptr, d, causal, scale, mode, stream);
}

int attn_bwd_gqa(const void* q, const void* k, const void* v, const void* o, const void* dO, const float* lse,
                 void* dq, void* dk, void* dv, float* delta, void* workspace, size_t workspace_bytes,
                 int B, int H, int H_kv, int N, int d, int causal, float scale, int mode, void* stream)
{
    return bwd_stage_impl(ATTN_BWD_STAGE_ALL, q, k, v, o, dO, lse, dq, dk, dv, delta, workspace, workspace_bytes,
                          B, H, H_kv, N, N, nullptr, d, causal, scale, mode, stream);
}

int attn_fwd_padded(const void* q, const void* k, const void* v, void* o, float* lse,
                    int B, int H, int H_kv, int N, int seqlen, int d, int causal, float scale, int mode, void* stream)
{
    return fwd_impl(q, k, v, o, lse, nullptr, B, H, H_kv, N, seqlen, nullptr, d, causal, scale, mode, stream);
}

int attn_bwd_padded(const void* q, const void* k, const void* v, const void* o, const void* dO, const float* lse,
                    void* dq, void* dk, void* dv, float* delta, void* workspace, size_t workspace_bytes,
                    int B, int H, int H_kv, int N, int seqlen, int d, int causal, float scale, int mode, void* stream)
{
    return bwd_stage_impl(ATTN_BWD_STAGE_ALL, q, k, v, o, dO, lse, dq, dk, dv, delta, workspace, workspace_bytes,
                          B, H, H_kv, N, seqlen, nullptr, d, causal, scale, mode, stream);
}

int attn_fwd_varlen(const void* q, const void* k, const void* v, void* o, float* lse, const int* seqlens,
                    int B, int H, int H_kv, int N, int d, int causal, float scale, int mode, void* stream)
{
    if (!seqlens) return ATTN_ERR_NULL;
    return fwd_impl(q, k, v, o, lse, nullptr, B, H, H_kv, N, N, seqlens, d, causal, scale, mode, stream);
}

int attn_bwd_varlen(const void* q, const void* k, const void* v, const void* o, const void* dO, const float* lse,
                    void* dq, void* dk, void* dv, float* delta, void* workspace, size_t workspace_bytes,
                    const int* seqlens, int B, int H, int H_kv, int N, int d, int causal, float scale, int mode,
                    void* stream)
{
    if (!seqlens) return ATTN_ERR_NULL;
    return bwd_stage_impl(ATTN_BWD_STAGE_ALL, q, k, v, o, dO, lse, dq, dk, dv, delta, workspace, workspace_bytes,
                          B, H, H_kv, N, N, seqlens, d, causal, scale, mode, stream);
}

// ---------------------------------------------------------------- packed variable-length batches
// The packed entry points copy between the caller's packed tensors and padded tensors in the workspace and run the
// per-batch-length kernels on those.  Layout of the workspace (every part a multiple of 256 bytes):
//   seqlens int[B] | q | k | v | o | lse            (forward)
//   ... | dO | dq | dk | dv | delta | FP32 dQ accumulator of attn_bwd_workspace_bytes(B, H, N_max, d)   (backward)
extern "C++" {
namespace {
struct PackedLayout {
    size_t seqlens, q, k, v, o, lse, dO, dq, dk, dv, delta, acc, total_fwd, total_bwd;
};
size_t round256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }
PackedLayout packed_layout(int B, int H, int Hkv, int N, int d)
{
    PackedLayout L;
    const size_t eq = round256(static_cast<size_t>(B) * H * N * d * 2), ekv = round256(static_cast<size_t>(B) * Hkv * N * d * 2);
    const size_t vec = round256(static_cast<size_t>(B) * H * N * 4);
    size_t p = 0;
    L.seqlens = p; p += round256(static_cast<size_t>(B) * 4);
    L.q = p; p += eq;
    L.k = p; p += ekv;
    L.v = p; p += ekv;
    L.o = p; p += eq;
    L.lse = p; p += vec;
    L.total_fwd = p;
    L.dO = p; p += eq;
    L.dq = p; p += eq;
    L.dk = p; p += ekv;
    L.dv = p; p += ekv;
    L.delta = p; p += vec;
    L.acc = p; p += round256(attn_bwd_workspace_bytes(B, H, N, d));
    L.total_bwd = p;
    return L;
}
int check_packed(const int* cu, void* workspace, int B, int H, int Hkv, int T, int N, int d)
{
    if (!cu) return ATTN_ERR_NULL;
    if (int e = check_shape(B, H, N, d)) return e;
    if (Hkv < 1 || H % Hkv != 0 || T < 1) return ATTN_ERR_SHAPE;
    if (static_cast<long long>(T) * H >= (1ll << 31)) return ATTN_ERR_SHAPE;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return ATTN_ERR_WORKSPACE;
    return ATTN_OK;
}
template <bool TO_PADDED>
int copy_rows(void* padded, const void* packed, const int* cu, int B, int Hx, int N, int d, cudaStream_t st)
{
    const int cpr = d / 8;
    const long long n = static_cast<long long>(B) * Hx * N * cpr;
    attn::packed_rows_kernel<TO_PADDED><<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(
        static_cast<uint4*>(padded), static_cast<uint4*>(const_cast<void*>(packed)), cu, Hx, N, cpr, n);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}
template <bool TO_PADDED>
int copy_vec(float* padded, const float* packed, const int* cu, int B, int H, int N, int T, cudaStream_t st)
{
    const long long n = static_cast<long long>(B) * H * N;
    attn::packed_vec_kernel<TO_PADDED><<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(
        padded, const_cast<float*>(packed), cu, H, N, T, n);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}
}  // namespace
}  // extern "C++"

size_t attn_packed_workspace_bytes(int B, int H, int H_kv, int N_max, int d, int backward)
{
    if (check_shape(B, H, N_max, d) != ATTN_OK || H_kv < 1 || H % H_kv != 0) return 0;
    const PackedLayout L = packed_layout(B, H, H_kv, N_max, d);
    return backward ? L.total_bwd : L.total_fwd;
}

int attn_fwd_packed(const void* q, const void* k, const void* v, void* o, float* lse, const int* cu_seqlens,
                    void* workspace, size_t workspace_bytes, int B, int H, int H_kv, int T, int N_max, int d,
                    int causal, float scale, int mode, void* stream)
{
    if (!q || !k || !v || !o || !lse) return ATTN_ERR_NULL;
    if (int e = check_packed(cu_seqlens, workspace, B, H, H_kv, T, N_max, d)) return e;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return ATTN_ERR_ALIGN;
    const PackedLayout L = packed_layout(B, H, H_kv, N_max, d);
    if (workspace_bytes < L.total_fwd) return ATTN_ERR_WORKSPACE;
    if (int e = check_device()) return e;
    uint8_t* w = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* seqlens = reinterpret_cast<int*>(w + L.seqlens);
    attn::packed_seqlens_kernel<<<(B + 127) / 128, 128, 0, st>>>(cu_seqlens, seqlens, B, N_max);
    if (cudaGetLastError() != cudaSuccess) return ATTN_ERR_CUDA;
    if (int e = copy_rows<true>(w + L.q, q, cu_seqlens, B, H, N_max, d, st)) return e;
    if (int e = copy_rows<true>(w + L.k, k, cu_seqlens, B, H_kv, N_max, d, st)) return e;
    if (int e = copy_rows<true>(w + L.v, v, cu_seqlens, B, H_kv, N_max, d, st)) return e;
    if (int e = fwd_impl(w + L.q, w + L.k, w + L.v, w + L.o, reinterpret_cast<float*>(w + L.lse), nullptr, B, H, H_kv,
                         N_max, N_max, seqlens, d, causal, scale, mode, stream))
        return e;
    if (int e = copy_rows<false>(w + L.o, o, cu_seqlens, B, H, N_max, d, st)) return e;
    return copy_vec<false>(reinterpret_cast<float*>(w + L.lse), lse, cu_seqlens, B, H, N_max, T, st);
}

int attn_bwd_packed(const void* q, const void* k, const void* v, const void* o, const void* dO, const float* lse,
                    void* dq, void* dk, void* dv, float* delta, const int* cu_seqlens,
                    void* workspace, size_t workspace_bytes, int B, int H, int H_kv, int T, int N_max, int d,
                    int causal, float scale, int mode, void* stream)
{
    if (!q || !k || !v || !o || !dO || !lse || !dq || !dk || !dv || !delta) return ATTN_ERR_NULL;
    if (int e = check_packed(cu_seqlens, workspace, B, H, H_kv, T, N_max, d)) return e;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(dO) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv))
        return ATTN_ERR_ALIGN;
    const PackedLayout L = packed_layout(B, H, H_kv, N_max, d);
    if (workspace_bytes < L.total_bwd) return ATTN_ERR_WORKSPACE;
    if (int e = check_device()) return e;
    uint8_t* w = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* seqlens = reinterpret_cast<int*>(w + L.seqlens);
    float* lse_p = reinterpret_cast<float*>(w + L.lse);
    float* delta_p = reinterpret_cast<float*>(w + L.delta);
    const bool given = (mode & ATTN_MODE_FLAG_DELTA_GIVEN) != 0;
    attn::packed_seqlens_kernel<<<(B + 127) / 128, 128, 0, st>>>(cu_seqlens, seqlens, B, N_max);
    if (cudaGetLastError() != cudaSuccess) return ATTN_ERR_CUDA;
    if (int e = copy_rows<true>(w + L.q, q, cu_seqlens, B, H, N_max, d, st)) return e;
    if (int e = copy_rows<true>(w + L.k, k, cu_seqlens, B, H_kv, N_max, d, st)) return e;
    if (int e = copy_rows<true>(w + L.v, v, cu_seqlens, B, H_kv, N_max, d, st)) return e;
    if (int e = copy_rows<true>(w + L.o, o, cu_seqlens, B, H, N_max, d, st)) return e;
    if (int e = copy_rows<true>(w + L.dO, dO, cu_seqlens, B, H, N_max, d, st)) return e;
    if (int e = copy_vec<true>(lse_p, lse, cu_seqlens, B, H, N_max, T, st)) return e;
    if (given)
        if (int e = copy_vec<true>(delta_p, delta, cu_seqlens, B, H, N_max, T, st)) return e;
    if (int e = bwd_stage_impl(ATTN_BWD_STAGE_ALL, w + L.q, w + L.k, w + L.v, w + L.o, w + L.dO, lse_p, w + L.dq, w + L.dk,
                               w + L.dv, delta_p, w + L.acc, L.total_bwd - L.acc, B, H, H_kv, N_max, N_max, seqlens, d,
                               causal, scale, mode, stream))
        return e;
    if (int e = copy_rows<false>(w + L.dq, dq, cu_seqlens, B, H, N_max, d, st)) return e;
    if (int e = copy_rows<false>(w + L.dk, dk, cu_seqlens, B, H_kv, N_max, d, st)) return e;
    if (int e = copy_rows<false>(w + L.dv, dv, cu_seqlens, B, H_kv, N_max, d, st)) return e;
    if (!given)
        if (int e = copy_vec<false>(delta_p, delta, cu_seqlens, B, H, N_max, T, st)) return e;
    return ATTN_OK;
}

int attn_bwd(const void* q, const void* k, const void* v, const void* o, const void* dO, const float* lse,
             void* dq, void* dk, void* dv, float* delta, void* workspace, size_t workspace_bytes,
             int B, int H, int N, int d, int causal, float scale, int mode, void* stream)
{
    return attn_bwd_stage(ATTN_BWD_STAGE_ALL, q, k, v, o, dO, lse, dq, dk, dv, delta, workspace, workspace_bytes,
                          B, H, N, d, causal, scale, mode, stream);
}

int attn_bwd_static(const void* q, const void* k, const void* v, const void* o, const void* dO, const float* lse,
                    void* dq, void* dk, void* dv, float* delta,
                    int B, int H, int N, int d, int causal, float scale, int mode, void* stream)
{
    // same order of checks as attn_bwd: pointers, shape, then the scratch size
    if (!q || !k || !v || !o || !dO || !lse || !dq || !dk || !dv || !delta) return ATTN_ERR_NULL;
    if (int e = check_shape(B, H, N, d)) return e;
    const size_t need = attn_bwd_workspace_bytes(B, H, N, d);
    if (need > static_cast<size_t>(ATTN_BWD_STATIC_MAX_BYTES)) return ATTN_ERR_WORKSPACE;   // problem too large for the built-in scratch
    if (int e = check_device()) return e;
    // Set-up, once per device, with that device current: translate the symbol into the device
    // address of this device's copy of the array.  No memory is allocated here or anywhere below.
    static std::atomic<void*> scratch_addr[MAX_DEVICES];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return ATTN_ERR_CUDA;
    void* scratch = scratch_addr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        if (cudaGetSymbolAddress(&scratch, g_static_bwd_scratch) != cudaSuccess || !scratch) return ATTN_ERR_CUDA;
        scratch_addr[dev].store(scratch, std::memory_order_release);
    }
    // Same three kernels as attn_bwd; the first one clears the part of the scratch this call uses.
    return attn_bwd_stage(ATTN_BWD_STAGE_ALL, q, k, v, o, dO, lse, dq, dk, dv, delta, scratch,
                          static_cast<size_t>(ATTN_BWD_STATIC_MAX_BYTES), B, H, N, d, causal, scale, mode, stream);
}

int attn_get_tiles(int d, int* Br, int* Bc)
{
    if (d != 64 && d != 128) return ATTN_ERR_SHAPE;
    if (!Br || !Bc) return ATTN_ERR_NULL;
    *Br = attn::FwdCfg<64>::BR;
    *Bc = attn::FwdCfg<64>::BC;
    return ATTN_OK;
}

int attn_set_guard_max_shift(float max_shift)
{
    if (!(max_shift > 0.0f) || !isfinite(max_shift)) return ATTN_ERR_PARAM;
    g_guard_cap.store(max_shift);
    return ATTN_OK;
}

float attn_get_guard_max_shift(void) { return g_guard_cap.load(); }

int attn_set_mitigation(float beta, float eps)
{
    if (!(beta > 1.0f) || !isfinite(beta) || !(eps > 0.0f) || !isfinite(eps)) return ATTN_ERR_PARAM;
    g_beta.store(beta);
    g_eps.store(eps);
    return ATTN_OK;
}

int attn_get_mitigation(float* beta, float* eps)
{
    if (!beta || !eps) return ATTN_ERR_NULL;
    *beta = g_beta.load();
    *eps = g_eps.load();
    return ATTN_OK;
}

int attn_last_device_status(void* stream)
{
    (void)stream;
    if (int e = check_device()) return e;
    int flag = 0;
    if (cudaMemcpyFromSymbol(&flag, g_device_status, sizeof(int)) != cudaSuccess) return ATTN_ERR_CUDA;
    if (flag) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)) != cudaSuccess) return ATTN_ERR_CUDA;
        return flag == 1 ? ATTN_ERR_TIMEOUT : ATTN_ERR_CUDA;     // 2: a kernel found its shared-memory layout out of bounds
    }
    return ATTN_OK;
}

int attn_selftest_wait_timeout(void* stream)
{
    if (int e = check_device()) return e;
    int* status = status_ptr();
    if (!status) return ATTN_ERR_CUDA;
    attn::wait_timeout_selftest_kernel<1000000ull><<<1, 96, 0, static_cast<cudaStream_t>(stream)>>>(status);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

const char* attn_strerror(int code)
{
    switch (code) {
        case ATTN_OK: return "ok";
        case ATTN_ERR_NULL: return "a required pointer is NULL";
        case ATTN_ERR_SHAPE: return "unsupported shape (need d in {64,128}, N a multiple of 128, B,H >= 1)";
        case ATTN_ERR_MODE: return "mode holds a bit this entry point does not accept (0 or 1, plus the ATTN_MODE_FLAG_* it documents)";
        case ATTN_ERR_PARAM: return "parameter out of range (scale > 0, beta > 1, eps > 0, all finite)";
        case ATTN_ERR_WORKSPACE: return "workspace missing, not 256-byte aligned, or too small";
        case ATTN_ERR_CUDA: return "a CUDA call or kernel launch failed";
        case ATTN_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case ATTN_ERR_DEVICE: return "current device is not compute capability 10.x (sm_100a only)";
        case ATTN_ERR_ALIGN: return "a tensor base address is not 16-byte aligned";
        default: return "unknown error code";
    }
}

}  // extern "C"
