// Tensor-core (tcgen05 / TMEM / TMA) skinny GEMM: interface used by the host orchestration.
#pragma once
#include "poss_internal.cuh"

struct TcGemmPlanCache;
TcGemmPlanCache* tc_plan_cache_create();
void tc_plan_cache_destroy(TcGemmPlanCache*);
size_t tc_gemm_scratch_bytes();
// true when the tensor-core kernel covers this product (bf16, K and leading dimension multiples of 64, ...)
bool tc_gemm_supported(const GemmSegs& segs, int K, int ldx, int M);
void launch_gemm_tc(Launcher& L, TcGemmPlanCache* cache, const bf16* X, int ldx, int M, const GemmSegs& segs, int K,
                    const bf16* bias, const float* residual, int ldr, float* out, int ldo, void* scratch,
                    int32_t* status);
