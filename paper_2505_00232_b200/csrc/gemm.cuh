// Prefill kernel (placeholder while the decode path is brought up).
#pragma once
#include <cuda_runtime.h>
#include "../../include/qlinear.h"
#include "layout.h"

namespace ql {
struct GemmPlan { int32_t unused; };
inline ql_status gemm_plan(const Layout&, int, GemmPlan* p) { p->unused = 0; return QL_OK; }
inline ql_status gemm_forward(const Layout&, const GemmPlan&, const uint8_t*, const void*, void*, int, cudaStream_t, int, bool)
{
    return QL_ERR_UNSUPPORTED;
}
}  // namespace ql
