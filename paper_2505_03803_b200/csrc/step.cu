#include "../../include/rwkvq.h"
extern "C" {
size_t rwkvq_step_plan_bytes(const rwkvq_gemv_op*, int, int) { return 0; }
rwkvq_status rwkvq_step_plan(const rwkvq_gemv_op*, int, int, void*, size_t, void*) { return RWKVQ_EUNSUPPORTED; }
rwkvq_status rwkvq_step_run(const void*, size_t, void*) { return RWKVQ_EUNSUPPORTED; }
}
