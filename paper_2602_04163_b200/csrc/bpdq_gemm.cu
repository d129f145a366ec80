#include "bpdq_internal.h"
namespace bpdq {
bool gemm_supported(int, int, int, int) { return false; }
int launch_gemm(bpdq_handle_s*, const void*, void*, int, cudaStream_t) { return set_error(BPDQ_ERR_UNSUPPORTED, "gemm: not built"); }
}
