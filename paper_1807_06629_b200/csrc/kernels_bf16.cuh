// bf16-operand tensor-core path (placeholder until the tcgen05 kernels land).
#pragma once
#include "prsgd_common.cuh"
namespace prsgd {
inline int tc_create(prsgd_ctx*, std::string* err) { *err = "BF16 precision is not available in this build"; return PRSGD_ERR_STATE; }
inline void tc_destroy(prsgd_ctx*) {}
inline int tc_bind_data(prsgd_ctx*, std::string* err) { *err = "BF16 precision is not available in this build"; return PRSGD_ERR_STATE; }
inline int tc_step(prsgd_ctx*, int64_t, bool) { return PRSGD_ERR_STATE; }
}
