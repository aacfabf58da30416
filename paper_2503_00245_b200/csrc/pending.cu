// Entry points whose kernels are not written yet: they refuse, loudly, rather than fall back.
#include "common.cuh"
extern "C" {
int moe_offload_create(const moe_config*, int32_t, int32_t, const void* const*, void*, size_t, moe_offload**) { return MOE_ERR_UNSUPPORTED; }
int moe_offload_destroy(moe_offload*) { return MOE_ERR_UNSUPPORTED; }
int moe_offload_ensure(moe_offload*, int32_t, const int32_t*, int32_t, void*) { return MOE_ERR_UNSUPPORTED; }
int moe_offload_slot_table(moe_offload*, int32_t, const int32_t**) { return MOE_ERR_UNSUPPORTED; }
int moe_offload_resident(moe_offload*, int32_t, int32_t*) { return MOE_ERR_UNSUPPORTED; }
int moe_offload_stats(moe_offload*, uint64_t*, uint64_t*, uint64_t*) { return MOE_ERR_UNSUPPORTED; }
int moe_stack_decode_step(moe_offload*, moe_ctx*, const moe_weights*, float*, int32_t*, void*, size_t, void*) { return MOE_ERR_UNSUPPORTED; }
int moe_expert_replacements(const int32_t*, int32_t, int32_t, int32_t, int32_t, unsigned long long*, void*) { return MOE_ERR_UNSUPPORTED; }
}
