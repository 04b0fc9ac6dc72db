// Small device helpers shared by the kernel files: one warp-level MMA, bf16 packing, the fast
// transcendental instructions and shared-memory addressing.
#pragma once

#include <stdint.h>

namespace ckv {

// D = A * B + D for one m16n8k16 tile, bf16 operands, fp32 accumulators
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// two floats rounded to nearest even, `lo` in the low half of the word
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float tanh_fast(float x)
{
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Range checks of the debug build (-DCKV_BOUNDS, the stand-in for a memory checker where none can run): every
// index taken from the compressed cache, every unit, query / output / partial row and shared-memory offset a
// kernel computes is compared with its bound; a violation ORs kErrBounds into the context's error word
// (ckv_last_stat "device_errors") and the access is redirected to element 0 -- nothing traps, nothing faults.
// In the normal build CKV_CLAMP is the identity and costs nothing.
constexpr int kErrBounds = 32;
#ifdef CKV_BOUNDS
template <typename T, typename B>
__device__ __forceinline__ T ckv_clamp(T v, B bound, int* err)
{
    if (v >= (T)0 && v < (T)bound) return v;
    if (err) atomicOr(err, kErrBounds);
    return (T)0;
}
#define CKV_CLAMP(v, bound, err) ::ckv::ckv_clamp((v), (bound), (err))
#else
#define CKV_CLAMP(v, bound, err) (v)
#endif

}  // namespace ckv
