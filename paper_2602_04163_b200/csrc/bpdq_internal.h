// Internal declarations shared by the translation units of libbpdq (not part of the ABI).
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include "bpdq.h"

#if defined(__CUDACC__)
#define BPDQ_HD __host__ __device__ __forceinline__
#else
#define BPDQ_HD inline
#endif

namespace bpdq {

constexpr int kBlockCols = 128;   // columns covered by one 16-byte plane unit
constexpr int kUnitBytes = 16;

// Byte offset of the 16-byte unit of (block b, plane i (0-based), row r).
BPDQ_HD size_t plane_unit_offset(int64_t b, int i, int64_t r, int K, int64_t out) {
    return (size_t)(((b * K + i) * out + r) * kUnitBytes);
}
// Byte offset (inside the coefficient section) of coefficient i of (group G, row r).
BPDQ_HD size_t coef_offset(int64_t G, int i, int64_t r, int K, int64_t out) {
    return (size_t)(((G * (K + 1) + i) * out + r) * 2);
}
BPDQ_HD size_t planes_bytes(int64_t out, int64_t in, int K) { return (size_t)(out * in * K / 8); }
BPDQ_HD size_t coefs_bytes(int64_t out, int64_t in, int K, int64_t g) {
    return (size_t)(out * ((in + g - 1) / g) * (K + 1) * 2);   // ceil(in / g) groups: the last one may be short
}

bool shape_supported(int out, int in, int K, int group);
int set_error(int code, const char* fmt, ...);

// Opt-in to more than 48 KB of dynamic shared memory is a per-device attribute of a kernel: one record per kernel
// instantiation, indexed by device ordinal.  Setting the attribute twice is harmless, so concurrent first calls
// need no lock; the record only saves the runtime call on later launches.
constexpr int kMaxDevices = 64;
struct SmemOptin {
    int bytes[kMaxDevices];       // largest size opted in to on each device so far (zero-initialised as a static)
};
template <typename Kernel>
inline int ensure_smem_optin(Kernel kernel, SmemOptin& rec, int device, int bytes, const char* who) {
    if (device < 0 || device >= kMaxDevices) return set_error(BPDQ_ERR_UNSUPPORTED, "%s: device ordinal %d", who, device);
    if (__atomic_load_n(&rec.bytes[device], __ATOMIC_ACQUIRE) >= bytes) return BPDQ_OK;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return set_error(BPDQ_ERR_CUDA, "%s: shared memory opt-in: %s", who, cudaGetErrorString(e));
    __atomic_store_n(&rec.bytes[device], bytes, __ATOMIC_RELEASE);
    return BPDQ_OK;
}

}  // namespace bpdq

namespace bpdq {
// Last cut of a launch's task space led by a handle (the cut depends on the shapes only): linears, their
// (row groups, slices or column ranges), a key of the cost model, CTAs, first task of every CTA.  n == 0: none yet.
struct LaunchPlan {
    int n, cost, grid;
    int shape[BPDQ_BATCH_MAX][2];
    int t_begin[193];
};
}  // namespace bpdq

struct bpdq_handle_s {
    int out, in, K, group, max_M, device;
    int sm_count;
    int smem_optin;           // largest dynamic shared memory a CTA may opt in to
    uint8_t* d_blob;          // planes then coefficients
    int caller_blob;          // 1: d_blob belongs to the caller (bpdq_linear_noalloc), its contents may be recent
    size_t blob_bytes, planes_bytes;
    float* d_ws;              // binary32 row sums of the split over input slices (zero between calls)
    size_t ws_bytes;
    unsigned* d_counters;     // arrival counters per 128 rows (zero between calls)
    size_t n_counters;
    int* d_status;            // device status word
    void* d_xstage;           // staging for bpdq_linear_host
    void* d_ystage;
    int gemv_max_m;
    uint64_t launches;
    int few_max_m;            // largest M the dispatcher sends to the few-token kernel
    void* d_few_maps;         // device copy of the few-token kernel's two tensor maps (null: not available)
    int* d_perm;              // input-channel permutation: stored column j multiplies x[perm[j]] (null: identity)
    void* d_xperm;            // [max_M][in] gathered activations for the kernels that do not fold the permutation into their loads
    void* d_bias;             // binary16 [out], added to every output row before the rounding (null: none)
    // Tensor maps of the blob for the tensor-core kernel (planes, coefficients), encoded at the first launch.
    alignas(64) unsigned char gemm_maps[2][128];
    int gemm_maps_ready;
    bpdq::LaunchPlan plan[2]; // [0] look-up-table kernel, [1] few-token kernel
};

// Kernel launchers (each returns a BPDQ_* status; all asynchronous on `stream`).
namespace bpdq {
int launch_fill(bpdq_handle_s* h, uint64_t seed, cudaStream_t stream);
int launch_dequant(bpdq_handle_s* h, void* w, cudaStream_t stream);
int launch_gemv_simple(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream);
int launch_gemv(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream);
int launch_gemv_batch(bpdq_handle_s* const* hs, const void* const* xs, void* const* ys, int n, int M, cudaStream_t stream, bool pair = false);
int launch_gemm(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream);
int launch_wait_limit_probe(bpdq_handle_s* h, cudaStream_t stream);
int launch_gather_columns(bpdq_handle_s* h, const void* x, int M, cudaStream_t stream);   // x[m][perm[j]] -> d_xperm[m][j]
int launch_swiglu(const void* gate, const void* up, void* hout, size_t n, cudaStream_t stream);
int launch_gemv_mma(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream);
int launch_gemv_mma_batch(bpdq_handle_s* const* hs, const void* const* xs, void* const* ys, int n, int M, cudaStream_t stream, bool pair = false);
bool gemv_mma_supported(int out, int in, int K, int group);
int few_prepare(bpdq_handle_s* h);
size_t gemv_workspace_bytes(int out, int in, int K, int group, int max_M, int sm_count);
size_t gemv_counter_count(int out);
bool gemv_supported(int out, int in, int K, int group);
bool gemm_supported(int out, int in, int K, int group);
}  // namespace bpdq
