#include "../../include/rwkvq.h"
extern "C" {
size_t rwkvq_prefill_workspace_bytes(const rwkvq_desc*, int, int) { return 0; }
rwkvq_status rwkvq_gemm_prefill(const rwkvq_desc*, const void*, const rwkvq_desc*, const void*, const void*, const void*, int, void*, int, void*, size_t, void*) { return RWKVQ_EUNSUPPORTED; }
}
