#include "bpdq_internal.h"
namespace bpdq {
size_t gemv_workspace_bytes(int, int, int, int, int, int) { return 0; }
size_t gemv_counter_count(int) { return 0; }
bool gemv_supported(int, int, int, int) { return false; }
int launch_gemv(bpdq_handle_s*, const void*, void*, int, cudaStream_t) { return set_error(BPDQ_ERR_UNSUPPORTED, "gemv: not built"); }
}
