// C ABI entry points that own device state: create / destroy / dequant / linear and friends.
// Argument checks happen here; kernels live in their own translation units.
#include <cstdio>
#include <cstring>
#include <new>

#include "bpdq_internal.h"
#include "bpdq_finish.cuh"

#include <cuda_fp16.h>

using namespace bpdq;

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int cuda_fail(const char* what, cudaError_t e) {
    return set_error(BPDQ_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

void free_handle(bpdq_handle_s* h) {
    if (!h) return;
    if (h->d_blob) cudaFree(h->d_blob);
    if (h->d_ws) cudaFree(h->d_ws);
    if (h->d_counters) cudaFree(h->d_counters);
    if (h->d_status) cudaFree(h->d_status);
    if (h->d_xstage) cudaFree(h->d_xstage);
    if (h->d_ystage) cudaFree(h->d_ystage);
    if (h->d_few_maps) cudaFree(h->d_few_maps);
    if (h->d_perm) cudaFree(h->d_perm);
    if (h->d_xperm) cudaFree(h->d_xperm);
    if (h->d_bias) cudaFree(h->d_bias);
    delete h;
}

// Activations of up to BPDQ_BATCH_MAX linears from pinned host memory into the handles' staging buffers, one launch:
// the kernel reads the host buffers through their device-visible addresses, sixteen bytes per thread and access.
struct GatherParams {
    const uint4* src[BPDQ_BATCH_MAX];
    uint4* dst[BPDQ_BATCH_MAX];
    unsigned end16[BPDQ_BATCH_MAX];     // running end of every buffer, in 16-byte units
    int n;
};
__global__ void gather_kernel(const __grid_constant__ GatherParams p) {
    // the look-up-table kernel behind it may take the free SMs and request its first weights at once; it reads x only
    // after its own griddepcontrol.wait, i.e. after this kernel has finished
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const unsigned total = p.end16[p.n - 1];
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        int k = 0;
        while (i >= p.end16[k]) ++k;
        const unsigned j = i - (k ? p.end16[k - 1] : 0u);
        p.dst[k][j] = p.src[k][j];
    }
}

// Activations in stored-column order: dst[m][j] = src[m][perm[j]], eight columns (sixteen bytes) per thread.
__global__ void gather_columns_kernel(const __half* __restrict__ src, const int* __restrict__ perm, __half* __restrict__ dst,
                                      int M, int in) {
    const int chunks = in / 8;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < (long long)M * chunks; i += (long long)gridDim.x * blockDim.x) {
        const int m = (int)(i / chunks), c = (int)(i % chunks);
        const int4 p0 = *reinterpret_cast<const int4*>(perm + c * 8), p1 = *reinterpret_cast<const int4*>(perm + c * 8 + 4);
        const __half* row = src + (size_t)m * in;
        __align__(16) __half v[8] = {row[p0.x], row[p0.y], row[p0.z], row[p0.w], row[p1.x], row[p1.y], row[p1.z], row[p1.w]};
        *reinterpret_cast<uint4*>(dst + (size_t)m * in + c * 8) = *reinterpret_cast<const uint4*>(v);
    }
}

// h = silu(gate) * up on rounded binary16 inputs (the many-token path of bpdq_gate_up_swiglu), two values per thread.
__global__ void swiglu_kernel(const __half2* __restrict__ gate, const __half2* __restrict__ up, __half2* __restrict__ hout, size_t n2) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n2; i += (size_t)gridDim.x * blockDim.x) {
        const float2 g = __half22float2(gate[i]), u = __half22float2(up[i]);
        hout[i] = __floats2half2_rn(bpdq::silu_f32(g.x) * u.x, bpdq::silu_f32(g.y) * u.y);
    }
}

// Device-visible address of a pinned (page-locked) host buffer; null for pageable or foreign memory.
void* mapped_address(const void* host) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
}

// A handle's buffers live on the device that was current in bpdq_create; a launch under another current device
// would hand that device pointers it cannot use.
int check_device(const bpdq_handle_s* h, const char* who) {
    int dev = -1;
    const cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return set_error(BPDQ_ERR_CUDA, "%s: cudaGetDevice: %s", who, cudaGetErrorString(e));
    if (dev != h->device)
        return set_error(BPDQ_ERR_INVALID, "%s: the handle lives on device %d, the current device is %d", who, h->device, dev);
    return BPDQ_OK;
}

int check_linear_args(bpdq_handle_s* h, const void* x, void* y, int M, const char* who) {
    if (!h) return set_error(BPDQ_ERR_INVALID, "%s: null handle", who);
    if (M < 0 || M > h->max_M) return set_error(BPDQ_ERR_INVALID, "%s: M=%d outside [0, max_M=%d]", who, M, h->max_M);
    if (M == 0) return BPDQ_OK;
    if (!x || !y) return set_error(BPDQ_ERR_INVALID, "%s: null pointer", who);
    return check_device(h, who);
}

// Everything bpdq_linear_batch requires of its handles and of M (pointers are checked by the callers, which
// differ in where those pointers live).
int check_batch_handles(const bpdq_handle_t* hs, int n, int M, const char* who) {
    if (!hs) return set_error(BPDQ_ERR_INVALID, "%s: null array", who);
    if (n < 1 || n > BPDQ_BATCH_MAX) return set_error(BPDQ_ERR_INVALID, "%s: n=%d outside [1, %d]", who, n, BPDQ_BATCH_MAX);
    if (M < 0 || M > BPDQ_GEMV_MAX_M) return set_error(BPDQ_ERR_INVALID, "%s: M=%d outside [0, %d]", who, M, BPDQ_GEMV_MAX_M);
    for (int k = 0; k < n; ++k) {
        if (!hs[k]) return set_error(BPDQ_ERR_INVALID, "%s: null handle at %d", who, k);
        if (M > hs[k]->max_M) return set_error(BPDQ_ERR_INVALID, "%s: M=%d exceeds max_M=%d of linear %d", who, M, hs[k]->max_M, k);
        if (hs[k]->K != hs[0]->K || hs[k]->device != hs[0]->device)
            return set_error(BPDQ_ERR_INVALID, "%s: linear %d differs from linear 0 in K or device", who, k);
        if ((hs[k]->group == 64) != (hs[0]->group == 64))
            return set_error(BPDQ_ERR_INVALID, "%s: linear %d and linear 0 differ in having group 64", who, k);
        if (!gemv_supported(hs[k]->out, hs[k]->in, hs[k]->K, hs[k]->group))
            return set_error(BPDQ_ERR_UNSUPPORTED, "%s: look-up-table kernel does not cover linear %d (K=%d g=%d; packed weights must stay below 4 GB)", who, k, hs[k]->K, hs[k]->group);
        for (int j = 0; j < k; ++j)
            if (hs[j] == hs[k]) return set_error(BPDQ_ERR_INVALID, "%s: handle %d repeats handle %d", who, k, j);
    }
    return M == 0 ? BPDQ_OK : check_device(hs[0], who);
}

}  // namespace

extern "C" int bpdq_create(bpdq_handle_t* hp, int out, int in, int K, int group, const void* host_blob,
                           uint64_t seed, int max_M) {
    if (!hp) return set_error(BPDQ_ERR_INVALID, "bpdq_create: null handle pointer");
    *hp = nullptr;
    if (max_M < 1) return set_error(BPDQ_ERR_INVALID, "bpdq_create: max_M=%d must be >= 1", max_M);
    if (!shape_supported(out, in, K, group))
        return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_create: unsupported shape out=%d in=%d K=%d g=%d", out, in, K, group);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_create: no CUDA device (%s)", cudaGetErrorString(e));
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, dev);
    if (e != cudaSuccess) return cuda_fail("cudaGetDeviceProperties", e);
    if (prop.major != 10)
        return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_create: device is sm_%d%d, this library is built for sm_100a only",
                         prop.major, prop.minor);

    bpdq_handle_s* h = new (std::nothrow) bpdq_handle_s();
    if (!h) return set_error(BPDQ_ERR_ALLOC, "bpdq_create: host allocation failed");
    std::memset(h, 0, sizeof(*h));
    h->out = out; h->in = in; h->K = K; h->group = group; h->max_M = max_M; h->device = dev;
    h->sm_count = prop.multiProcessorCount;
    h->smem_optin = (int)prop.sharedMemPerBlockOptin;
    h->planes_bytes = planes_bytes(out, in, K);
    h->blob_bytes = h->planes_bytes + coefs_bytes(out, in, K, group);
    h->ws_bytes = gemv_workspace_bytes(out, in, K, group, max_M, h->sm_count);
    h->n_counters = gemv_counter_count(out);
    // Measured on 72B-shaped layers: one two-token pass of the look-up-table kernel (37 us on the largest projections)
    // beats every other kernel; a second pass (64 us) does not beat the few-token kernel.
    h->gemv_max_m = 2;
    // 3 to 16 tokens: the few-token kernel reads the weights once (43-60 us on the largest 72B-shaped projections
    // against 64 us for two look-up-table passes and 67-78 us for the tcgen05 tile kernel); from 17 tokens on its second
    // token tile costs more than the tile kernel.
    h->few_max_m = 16;
    // sixteen candidates (the few-token kernel then takes tasks of two row groups): 83-88 us on the largest projections for
    // 3 to 16 tokens against 77 / 92 us for two look-up-table passes at 3 / 4 tokens (103 / 120 us at g = 64) and 118 us
    // for the tile kernel
    if (K == 4) h->gemv_max_m = group == 64 ? 2 : 3;

    const size_t stage_x = (size_t)max_M * in * 2, stage_y = (size_t)max_M * out * 2;
    if ((e = cudaMalloc(&h->d_blob, h->blob_bytes)) != cudaSuccess ||
        (e = cudaMalloc(&h->d_ws, h->ws_bytes ? h->ws_bytes : 16)) != cudaSuccess ||
        (e = cudaMalloc(&h->d_counters, (h->n_counters ? h->n_counters : 1) * sizeof(unsigned))) != cudaSuccess ||
        (e = cudaMalloc(&h->d_status, sizeof(int))) != cudaSuccess ||
        (e = cudaMalloc(&h->d_xstage, stage_x)) != cudaSuccess ||
        (e = cudaMalloc(&h->d_ystage, stage_y)) != cudaSuccess) {
        free_handle(h);
        cudaGetLastError();
        return set_error(BPDQ_ERR_ALLOC, "bpdq_create: cudaMalloc failed (%s)", cudaGetErrorString(e));
    }
    cudaMemset(h->d_counters, 0, (h->n_counters ? h->n_counters : 1) * sizeof(unsigned));
    cudaMemset(h->d_status, 0, sizeof(int));
    cudaMemset(h->d_ws, 0, h->ws_bytes ? h->ws_bytes : 16);
    int rc = few_prepare(h);
    if (rc != BPDQ_OK) { free_handle(h); return rc; }
    if (host_blob) {
        e = cudaMemcpy(h->d_blob, host_blob, h->blob_bytes, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) rc = cuda_fail("bpdq_create: blob copy", e);
    } else {
        rc = launch_fill(h, seed, nullptr);
    }
    if (rc == BPDQ_OK) {
        e = cudaDeviceSynchronize();
        if (e != cudaSuccess) rc = cuda_fail("bpdq_create: synchronize", e);
    }
    if (rc != BPDQ_OK) { free_handle(h); return rc; }
    *hp = h;
    return BPDQ_OK;
}

extern "C" int bpdq_destroy(bpdq_handle_t h) {
    if (!h) return BPDQ_OK;
    cudaError_t e = cudaDeviceSynchronize();
    free_handle(h);
    if (e != cudaSuccess) return cuda_fail("bpdq_destroy: synchronize", e);
    return BPDQ_OK;
}

extern "C" int bpdq_dequant(bpdq_handle_t h, void* w, void* stream) {
    if (!h) return set_error(BPDQ_ERR_INVALID, "bpdq_dequant: null handle");
    if (!w) return set_error(BPDQ_ERR_INVALID, "bpdq_dequant: null output pointer");
    if (!aligned16(w)) return set_error(BPDQ_ERR_INVALID, "bpdq_dequant: output pointer not 16-byte aligned");
    if (const int rc = check_device(h, "bpdq_dequant"); rc != BPDQ_OK) return rc;
    return launch_dequant(h, w, static_cast<cudaStream_t>(stream));
}

extern "C" int bpdq_linear_ex(bpdq_handle_t h, const void* x, void* y, int M, int kernel, void* stream) {
    int rc = check_linear_args(h, x, y, M, "bpdq_linear");
    if (rc != BPDQ_OK || M == 0) return rc;
    if (!aligned16(x) || !aligned16(y))
        return set_error(BPDQ_ERR_INVALID, "bpdq_linear: x and y must be 16-byte aligned");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (kernel == BPDQ_KERNEL_AUTO) {
        const bool gv = gemv_supported(h->out, h->in, h->K, h->group);
        const bool gm = gemm_supported(h->out, h->in, h->K, h->group);
        const bool fw = gemv_mma_supported(h->out, h->in, h->K, h->group);
        if (gv && (M <= h->gemv_max_m || !gm) && M <= BPDQ_GEMV_MAX_M) kernel = BPDQ_KERNEL_GEMV;
        else if (fw && M <= h->few_max_m && M <= BPDQ_FEW_MAX_M) kernel = BPDQ_KERNEL_FEW;
        else if (gm) kernel = BPDQ_KERNEL_GEMM;
        else kernel = BPDQ_KERNEL_GEMV_SIMPLE;
    }
    if (h->d_perm && kernel != BPDQ_KERNEL_GEMV) {
        // only the look-up-table kernel reads x through the permutation; the others get a gathered copy
        if (x == h->d_xperm) return set_error(BPDQ_ERR_INVALID, "bpdq_linear: x aliases the handle's gather buffer");
        if (const int rc = launch_gather_columns(h, x, M, s); rc != BPDQ_OK) return rc;
        x = h->d_xperm;
    }
    switch (kernel) {
        case BPDQ_KERNEL_GEMV:
            if (M > BPDQ_GEMV_MAX_M)
                return set_error(BPDQ_ERR_INVALID, "bpdq_linear: look-up-table kernel takes M <= %d, got %d", BPDQ_GEMV_MAX_M, M);
            if (!gemv_supported(h->out, h->in, h->K, h->group))
                return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_linear: look-up-table kernel does not cover this linear (K=%d g=%d; packed weights must stay below 4 GB)", h->K, h->group);
            return launch_gemv(h, x, y, M, s);
        case BPDQ_KERNEL_GEMM:
            if (!gemm_supported(h->out, h->in, h->K, h->group))
                return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_linear: tensor-core kernel does not cover K=%d g=%d", h->K, h->group);
            return launch_gemm(h, x, y, M, s);
        case BPDQ_KERNEL_GEMV_SIMPLE:
            return launch_gemv_simple(h, x, y, M, s);
        case BPDQ_KERNEL_FEW:
            if (M > BPDQ_FEW_MAX_M)
                return set_error(BPDQ_ERR_INVALID, "bpdq_linear: few-token kernel takes M <= %d, got %d", BPDQ_FEW_MAX_M, M);
            if (!gemv_mma_supported(h->out, h->in, h->K, h->group))
                return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_linear: few-token kernel does not cover this linear (K=%d g=%d)", h->K, h->group);
            return launch_gemv_mma(h, x, y, M, s);
        default:
            return set_error(BPDQ_ERR_INVALID, "bpdq_linear: unknown kernel id %d", kernel);
    }
}

extern "C" int bpdq_linear_batch(const bpdq_handle_t* hs, const void* const* xs, void* const* ys, int n, int M, void* stream) {
    if (!hs || !xs || !ys) return set_error(BPDQ_ERR_INVALID, "bpdq_linear_batch: null array");
    if (const int rc = check_batch_handles(hs, n, M, "bpdq_linear_batch"); rc != BPDQ_OK) return rc;
    if (M == 0) return BPDQ_OK;
    for (int k = 0; k < n; ++k)
        if (!xs[k] || !ys[k] || !aligned16(xs[k]) || !aligned16(ys[k]))
            return set_error(BPDQ_ERR_INVALID, "bpdq_linear_batch: x and y of linear %d must be non-null and 16-byte aligned", k);
    // above the look-up-table threshold the few-token kernel takes the whole batch, when every linear allows it
    bool few = M > hs[0]->gemv_max_m && M <= hs[0]->few_max_m && M <= BPDQ_FEW_MAX_M;
    for (int k = 0; few && k < n; ++k)
        few = hs[k]->d_few_maps && gemv_mma_supported(hs[k]->out, hs[k]->in, hs[k]->K, hs[k]->group) &&
              (size_t)M * hs[k]->out * sizeof(float) <= hs[k]->ws_bytes;
    if (few) {
        const void* xg[BPDQ_BATCH_MAX];
        for (int k = 0; k < n; ++k) {
            xg[k] = xs[k];
            if (hs[k]->d_perm) {
                if (const int rc = launch_gather_columns(hs[k], xs[k], M, static_cast<cudaStream_t>(stream)); rc != BPDQ_OK) return rc;
                xg[k] = hs[k]->d_xperm;
            }
        }
        return launch_gemv_mma_batch(hs, xg, ys, n, M, static_cast<cudaStream_t>(stream));
    }
    return launch_gemv_batch(hs, xs, ys, n, M, static_cast<cudaStream_t>(stream));
}

extern "C" int bpdq_linear(bpdq_handle_t h, const void* x, void* y, int M, void* stream) {
    return bpdq_linear_ex(h, x, y, M, BPDQ_KERNEL_AUTO, stream);
}

extern "C" int bpdq_linear_host(bpdq_handle_t h, const void* x_host, void* y_host, int M, void* stream) {
    int rc = check_linear_args(h, x_host, y_host, M, "bpdq_linear_host");
    if (rc != BPDQ_OK || M == 0) return rc;
    if (M <= h->gemv_max_m && M <= BPDQ_GEMV_MAX_M && gemv_supported(h->out, h->in, h->K, h->group))
        return bpdq_linear_batch_host(&h, &x_host, &y_host, 1, M, stream);      // the look-up-table kernel: same path as a batch of one
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(h->d_xstage, x_host, (size_t)M * h->in * 2, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail("bpdq_linear_host: copy in", e);
    rc = bpdq_linear_ex(h, h->d_xstage, h->d_ystage, M, BPDQ_KERNEL_AUTO, stream);
    if (rc != BPDQ_OK) return rc;
    e = cudaMemcpyAsync(y_host, h->d_ystage, (size_t)M * h->out * 2, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail("bpdq_linear_host: copy out", e);
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail("bpdq_linear_host: synchronize", e);
    return BPDQ_OK;
}

extern "C" int bpdq_linear_batch_host(const bpdq_handle_t* hs, const void* const* xs_host, void* const* ys_host, int n, int M,
                                      void* stream) {
    if (!hs || !xs_host || !ys_host) return set_error(BPDQ_ERR_INVALID, "bpdq_linear_batch_host: null array");
    // every rule of bpdq_linear_batch is checked before anything is enqueued
    if (const int rc = check_batch_handles(hs, n, M, "bpdq_linear_batch_host"); rc != BPDQ_OK) return rc;
    if (M == 0) return BPDQ_OK;
    for (int k = 0; k < n; ++k)
        if (!xs_host[k] || !ys_host[k]) return set_error(BPDQ_ERR_INVALID, "bpdq_linear_batch_host: null pointer at %d", k);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const void* xd[BPDQ_BATCH_MAX];
    void* yd[BPDQ_BATCH_MAX];
    // Pinned, 16-byte aligned host buffers: one gather launch brings every x into its staging buffer, and the kernel
    // writes every y straight into host memory (its stores are posted, nobody waits for them), so a step is two
    // launches and one wait instead of 2n copies.  Anything else takes the copy path below.
    {
        GatherParams g;
        g.n = n;
        bool direct = true;
        unsigned end16 = 0;
        for (int k = 0; k < n && direct; ++k) {
            void* xm = mapped_address(xs_host[k]);
            void* ym = mapped_address(ys_host[k]);
            direct = xm && ym && aligned16(xm) && aligned16(ym);
            g.src[k] = static_cast<const uint4*>(xm);
            g.dst[k] = static_cast<uint4*>(hs[k]->d_xstage);
            end16 += (unsigned)((size_t)M * hs[k]->in * 2 / 16);        // in is a multiple of 128: whole 16-byte units
            g.end16[k] = end16;
            xd[k] = hs[k]->d_xstage;
            yd[k] = ym;
        }
        if (direct) {
            // few, full CTAs: every thread has about one access in flight, and most SMs stay free for the kernel behind
            unsigned blocks = (end16 + 1023u) / 1024u;
            if (blocks > 64u) blocks = 64u;
            gather_kernel<<<blocks, 1024, 0, s>>>(g);
            cudaError_t e = cudaGetLastError();
            if (e != cudaSuccess) return cuda_fail("bpdq_linear_batch_host: gather launch", e);
            hs[0]->launches += 1;
            const int rc = bpdq_linear_batch(hs, xd, yd, n, M, stream);
            if (rc != BPDQ_OK) return rc;
            e = cudaStreamSynchronize(s);
            if (e != cudaSuccess) return cuda_fail("bpdq_linear_batch_host: synchronize", e);
            return BPDQ_OK;
        }
    }
    for (int k = 0; k < n; ++k) {
        cudaError_t e = cudaMemcpyAsync(hs[k]->d_xstage, xs_host[k], (size_t)M * hs[k]->in * 2, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return cuda_fail("bpdq_linear_batch_host: copy in", e);
        xd[k] = hs[k]->d_xstage;
        yd[k] = hs[k]->d_ystage;
    }
    int rc = bpdq_linear_batch(hs, xd, yd, n, M, stream);
    if (rc != BPDQ_OK) return rc;
    for (int k = 0; k < n; ++k) {
        cudaError_t e = cudaMemcpyAsync(ys_host[k], hs[k]->d_ystage, (size_t)M * hs[k]->out * 2, cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return cuda_fail("bpdq_linear_batch_host: copy out", e);
    }
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail("bpdq_linear_batch_host: synchronize", e);
    return BPDQ_OK;
}

extern "C" int bpdq_set_gemv_max_m(bpdq_handle_t h, int max_gemv_m) {
    if (!h) return set_error(BPDQ_ERR_INVALID, "bpdq_set_gemv_max_m: null handle");
    if (max_gemv_m < 0 || max_gemv_m > BPDQ_GEMV_MAX_M)
        return set_error(BPDQ_ERR_INVALID, "bpdq_set_gemv_max_m: %d outside [0, %d]", max_gemv_m, BPDQ_GEMV_MAX_M);
    h->gemv_max_m = max_gemv_m;
    return BPDQ_OK;
}

extern "C" int bpdq_set_few_max_m(bpdq_handle_t h, int max_few_m) {
    if (!h) return set_error(BPDQ_ERR_INVALID, "bpdq_set_few_max_m: null handle");
    if (max_few_m < 0 || max_few_m > BPDQ_FEW_MAX_M)
        return set_error(BPDQ_ERR_INVALID, "bpdq_set_few_max_m: %d outside [0, %d]", max_few_m, BPDQ_FEW_MAX_M);
    h->few_max_m = max_few_m;
    return BPDQ_OK;
}

extern "C" int bpdq_read_blob(bpdq_handle_t h, void* host_blob) {
    if (!h || !host_blob) return set_error(BPDQ_ERR_INVALID, "bpdq_read_blob: null pointer");
    if (const int rc = check_device(h, "bpdq_read_blob"); rc != BPDQ_OK) return rc;
    cudaError_t e = cudaMemcpy(host_blob, h->d_blob, h->blob_bytes, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail("bpdq_read_blob", e);
    return BPDQ_OK;
}

extern "C" int bpdq_get_status(bpdq_handle_t h, void* stream) {
    if (!h) return set_error(BPDQ_ERR_INVALID, "bpdq_get_status: null handle");
    if (const int rc = check_device(h, "bpdq_get_status"); rc != BPDQ_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int st = 0;
    cudaError_t e = cudaMemcpyAsync(&st, h->d_status, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(h->d_status, 0, sizeof(int), s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail("bpdq_get_status", e);
    if (st != BPDQ_OK) return set_error(st, "a device-side bounded wait expired (status %d)", st);
    return BPDQ_OK;
}

extern "C" int bpdq_probe_wait_limit(bpdq_handle_t h, void* stream) {
    if (!h) return set_error(BPDQ_ERR_INVALID, "bpdq_probe_wait_limit: null handle");
    if (const int rc = check_device(h, "bpdq_probe_wait_limit"); rc != BPDQ_OK) return rc;
    return launch_wait_limit_probe(h, static_cast<cudaStream_t>(stream));
}

extern "C" int bpdq_launch_count(bpdq_handle_t h, uint64_t* count) {
    if (!h || !count) return set_error(BPDQ_ERR_INVALID, "bpdq_launch_count: null pointer");
    *count = h->launches;
    return BPDQ_OK;
}

namespace bpdq {

int launch_gather_columns(bpdq_handle_s* h, const void* x, int M, cudaStream_t stream) {
    const long long items = (long long)M * (h->in / 8);
    long long blocks = (items + 255) / 256;
    if (blocks > 4LL * h->sm_count) blocks = 4LL * h->sm_count;
    gather_columns_kernel<<<(unsigned)blocks, 256, 0, stream>>>(static_cast<const __half*>(x), h->d_perm, static_cast<__half*>(h->d_xperm), M, h->in);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_error(BPDQ_ERR_CUDA, "gather launch: %s", cudaGetErrorString(e));
    h->launches += 1;
    return BPDQ_OK;
}

int launch_swiglu(const void* gate, const void* up, void* hout, size_t n, cudaStream_t stream) {
    const size_t n2 = n / 2;                                      // out is a multiple of 16: an even count
    size_t blocks = (n2 + 255) / 256;
    if (blocks > 1184) blocks = 1184;
    swiglu_kernel<<<(unsigned)blocks, 256, 0, stream>>>(static_cast<const __half2*>(gate), static_cast<const __half2*>(up), static_cast<__half2*>(hout), n2);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_error(BPDQ_ERR_CUDA, "gated unit launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

}  // namespace bpdq

extern "C" int bpdq_set_input_permutation(bpdq_handle_t h, const int32_t* perm) {
    if (!h) return set_error(BPDQ_ERR_INVALID, "bpdq_set_input_permutation: null handle");
    if (const int rc = check_device(h, "bpdq_set_input_permutation"); rc != BPDQ_OK) return rc;
    cudaError_t e = cudaDeviceSynchronize();                      // nothing in flight may still read the old permutation
    if (e != cudaSuccess) return cuda_fail("bpdq_set_input_permutation: synchronize", e);
    if (!perm) {
        if (h->d_perm) cudaFree(h->d_perm);
        if (h->d_xperm) cudaFree(h->d_xperm);
        h->d_perm = nullptr; h->d_xperm = nullptr;
        return BPDQ_OK;
    }
    {
        unsigned char* seen = new (std::nothrow) unsigned char[h->in]();
        if (!seen) return set_error(BPDQ_ERR_ALLOC, "bpdq_set_input_permutation: host allocation failed");
        bool ok = true;
        for (int j = 0; j < h->in && ok; ++j) {
            ok = perm[j] >= 0 && perm[j] < h->in && !seen[perm[j]];
            if (ok) seen[perm[j]] = 1;
        }
        delete[] seen;
        if (!ok) return set_error(BPDQ_ERR_INVALID, "bpdq_set_input_permutation: not a permutation of 0..%d", h->in - 1);
    }
    if (!h->d_perm && (e = cudaMalloc(&h->d_perm, (size_t)h->in * sizeof(int))) != cudaSuccess) {
        h->d_perm = nullptr;
        return set_error(BPDQ_ERR_ALLOC, "bpdq_set_input_permutation: cudaMalloc failed (%s)", cudaGetErrorString(e));
    }
    if (!h->d_xperm && (e = cudaMalloc(&h->d_xperm, (size_t)h->max_M * h->in * 2)) != cudaSuccess) {
        cudaFree(h->d_perm);
        h->d_perm = nullptr; h->d_xperm = nullptr;
        return set_error(BPDQ_ERR_ALLOC, "bpdq_set_input_permutation: cudaMalloc failed (%s)", cudaGetErrorString(e));
    }
    e = cudaMemcpy(h->d_perm, perm, (size_t)h->in * sizeof(int), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) return cuda_fail("bpdq_set_input_permutation: copy", e);
    return BPDQ_OK;
}

extern "C" int bpdq_set_bias(bpdq_handle_t h, const uint16_t* bias) {
    if (!h) return set_error(BPDQ_ERR_INVALID, "bpdq_set_bias: null handle");
    if (const int rc = check_device(h, "bpdq_set_bias"); rc != BPDQ_OK) return rc;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail("bpdq_set_bias: synchronize", e);
    if (!bias) {
        if (h->d_bias) cudaFree(h->d_bias);
        h->d_bias = nullptr;
        return BPDQ_OK;
    }
    if (!h->d_bias && (e = cudaMalloc(&h->d_bias, (size_t)h->out * 2)) != cudaSuccess) {
        h->d_bias = nullptr;
        return set_error(BPDQ_ERR_ALLOC, "bpdq_set_bias: cudaMalloc failed (%s)", cudaGetErrorString(e));
    }
    e = cudaMemcpy(h->d_bias, bias, (size_t)h->out * 2, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) return cuda_fail("bpdq_set_bias: copy", e);
    return BPDQ_OK;
}

extern "C" int bpdq_gate_up_swiglu(bpdq_handle_t hg, bpdq_handle_t hu, const void* x, void* hout, int M, void* stream) {
    if (!hg || !hu) return set_error(BPDQ_ERR_INVALID, "bpdq_gate_up_swiglu: null handle");
    if (hg == hu) return set_error(BPDQ_ERR_INVALID, "bpdq_gate_up_swiglu: gate and up are the same handle");
    if (hg->out != hu->out || hg->in != hu->in || hg->K != hu->K || hg->device != hu->device)
        return set_error(BPDQ_ERR_INVALID, "bpdq_gate_up_swiglu: gate and up differ in shape, K or device");
    if (M < 0 || M > hg->max_M || M > hu->max_M) return set_error(BPDQ_ERR_INVALID, "bpdq_gate_up_swiglu: M=%d outside [0, max_M]", M);
    if (M == 0) return BPDQ_OK;
    if (!x || !hout || !aligned16(x) || !aligned16(hout))
        return set_error(BPDQ_ERR_INVALID, "bpdq_gate_up_swiglu: x and h must be non-null and 16-byte aligned");
    if (const int rc = check_device(hg, "bpdq_gate_up_swiglu"); rc != BPDQ_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    bpdq_handle_s* hs[2] = {hg, hu};
    const bool same_g64 = (hg->group == 64) == (hu->group == 64);
    const bool lut = same_g64 && M <= hg->gemv_max_m && M <= BPDQ_GEMV_MAX_M && gemv_supported(hg->out, hg->in, hg->K, hg->group) &&
                     gemv_supported(hu->out, hu->in, hu->K, hu->group);
    bool few = same_g64 && !lut && M <= hg->few_max_m && M <= BPDQ_FEW_MAX_M && hg->d_few_maps && hu->d_few_maps &&
               (size_t)M * hg->out * sizeof(float) <= hg->ws_bytes && (size_t)M * hu->out * sizeof(float) <= hu->ws_bytes;
    if (lut || few) {
        // one launch over both linears; the kernel that completes a block of rows applies the unit
        const void* xs[2] = {x, x};
        if (few) {                                                 // this kernel does not read through a permutation: gather first
            for (int k = 0; k < 2; ++k) {
                if (hs[k]->d_perm) {
                    if (const int rc = launch_gather_columns(hs[k], x, M, s); rc != BPDQ_OK) return rc;
                    xs[k] = hs[k]->d_xperm;
                }
            }
        }
        void* ys[2] = {hout, hout};
        return lut ? launch_gemv_batch(hs, xs, ys, 2, M, s, true) : launch_gemv_mma_batch(hs, xs, ys, 2, M, s, true);
    }
    // many tokens: both projections through the dispatcher into the handles' own output buffers, then the unit
    for (int k = 0; k < 2; ++k)
        if (const int rc = bpdq_linear_ex(hs[k], x, hs[k]->d_ystage, M, BPDQ_KERNEL_AUTO, stream); rc != BPDQ_OK) return rc;
    hg->launches += 1;
    return launch_swiglu(hg->d_ystage, hu->d_ystage, hout, (size_t)M * hg->out, s);
}
