#include "../../include/rwkvq.h"
extern "C" {
size_t rwkvq_proxy_workspace_bytes(int) { return 0; }
rwkvq_status rwkvq_proxy_select(const void* const*, const int*, const int*, int, int, double, double, double*, double*, int*, void*, size_t, void*) { return RWKVQ_EUNSUPPORTED; }
}
