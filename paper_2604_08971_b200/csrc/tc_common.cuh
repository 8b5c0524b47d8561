// Pieces shared by the tcgen05 kernels (FFN pair, SentryAttend core): the GELU epilogue
// arithmetic, warp-level barrier helpers, single-lane election and the TMA tensor-map encoder.
#pragma once
#include <cuda.h>
#include <cuda_fp8.h>
#include <math.h>

#include "common.cuh"
#include "ptx/sm100.cuh"

namespace {

// gelu(z) = z/2 (1 + erf(z / sqrt 2)), with erf(z / sqrt 2) evaluated as tanh(z (c1 + c2 z^2)) on the
// hardware tanh (one special-function operation per element).  c1 = 0.7985835, c2 = 0.03538746:
// own fit that minimises the largest error relative to gelu(|z|) -- 1.5e-4 of gelu(|z|) for every
// z (checked against scipy.special.erf on 160 k points); the tanh unit adds at most 2^-11 of its
// result, i.e. 2.4e-4 |z|.  Both are more than ten times below the rounding of the bf16 value
// that is stored (2^-9 of it).  Both coefficients are positive, so z (c1 + c2 z^2) is monotone
// and saturates the tanh for large |z| without a clamp.
// Evaluated on two values at once with the packed fp32 instructions of sm_100 (two lanes of a
// 64-bit register per instruction), result rounded to a bf16 pair: 4.5 issue slots per element,
// which matters because the GELU epilogue is what the tensor pipe ends up waiting for.
__device__ __forceinline__ uint64_t f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// gelu of a pair by the tanh form above, as two floats
__device__ __forceinline__ void gelu_erf_fast_x2(float z0, float z1, float& g0, float& g1) {
    const uint64_t Z = f32x2(z0, z1), zero = f32x2(0.f, 0.f);
    const uint64_t Z2 = fma_f32x2(Z, Z, zero);
    const uint64_t P = fma_f32x2(Z2, f32x2(0.03538746f, 0.03538746f), f32x2(0.7985835f, 0.7985835f));
    const uint64_t U = fma_f32x2(P, Z, zero);
    float u0, u1, t0, t1;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(u0), "=f"(u1) : "l"(U));
    asm("tanh.approx.f32 %0, %1;" : "=f"(t0) : "f"(u0));
    asm("tanh.approx.f32 %0, %1;" : "=f"(t1) : "f"(u1));
    const uint64_t H = fma_f32x2(Z, f32x2(0.5f, 0.5f), zero);
    const uint64_t G = fma_f32x2(H, f32x2(t0, t1), H);
    asm("mov.b64 {%0, %1}, %2;" : "=f"(g0), "=f"(g1) : "l"(G));
}
__device__ __forceinline__ uint32_t gelu_erf_fast_bf16x2(float z0, float z1) {
    float g0, g1;
    gelu_erf_fast_x2(z0, z1, g0, g1);
    __nv_bfloat162 v = __floats2bfloat162_rn(g0, g1);
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}
// Two floats -> one 32-bit pair of the storage type (low half = a): bf16, or IEEE half when F16.
template <bool F16>
__device__ __forceinline__ uint32_t pack_16x2(float a, float b) {
    if constexpr (F16) {
        const __half2 v = __floats2half2_rn(a, b);
        return *reinterpret_cast<const uint32_t*>(&v);
    } else {
        return pack_bf16x2(a, b);
    }
}
// gelu of a pair, rounded to the storage type.  Both types take the tanh form: its error (1.5e-4
// of the value plus the tanh unit's 2^-11) is of the size of half's own rounding (2^-12 to 2^-11),
// and the erf of the math library costs five times the issue slots, which the epilogue -- the
// stage the tensor pipe waits for -- does not have (measured: 92 against 55 us on a D = 256 shape).
template <bool F16>
__device__ __forceinline__ uint32_t gelu_pack_16x2(float z0, float z1) {
    if constexpr (F16) {
        float g0, g1;
        gelu_erf_fast_x2(z0, z1, g0, g1);
        return pack_16x2<true>(g0, g1);
    } else {
        return gelu_erf_fast_bf16x2(z0, z1);
    }
}

// gelu of four values by the tanh form, times `post`, rounded to FP8 e4m3 (saturating at +-448) and
// packed low byte first.
__device__ __forceinline__ uint32_t gelu_pack_e4m3x4(float z0, float z1, float z2, float z3, float post) {
    float g0, g1, g2, g3;
    gelu_erf_fast_x2(z0, z1, g0, g1);
    gelu_erf_fast_x2(z2, z3, g2, g3);
    const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(g0 * post, g1 * post), __NV_SATFINITE, __NV_E4M3);
    const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(g2 * post, g3 * post), __NV_SATFINITE, __NV_E4M3);
    return lo | (hi << 16);
}

__device__ __forceinline__ void cp_async_wait_pending(int n) {
    if (n <= 0) ptx::cp_async_wait_group<0>();
    else if (n == 1) ptx::cp_async_wait_group<1>();
    else ptx::cp_async_wait_group<2>();
}

// Bounded wait by every lane of a warp; the result is the same in all lanes.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    const bool ok = ptx::mbar_wait(ptx::smem_u32(bar), parity, abort_flag);
    return __all_sync(0xffffffffu, ok);
}
// One arrival for the whole warp, after every lane has reached this point.
__device__ __forceinline__ void warp_arrive(uint64_t* bar) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) ptx::mbar_arrive(ptx::smem_u32(bar));
}

// One lane of a fully converged warp.  The single-thread instructions (TMA, UMMA, commit) are
// issued from inside `if (elect_one())` while the whole warp walks the schedule: operands
// computed by all lanes stay warp-uniform, which about halves the cost of issuing them
// compared with a lane-0 branch around the whole loop.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}


typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 row-major [rows, cols] -> 2-D map with a box of box_rows x box_cols elements whose rows
// are box_cols * 2 = 32, 64 or 128 bytes wide, swizzled with the mode of that width.
bool make_map_2d(CUtensorMap* tm, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows,
                 uint32_t box_cols) {
    EncodeTiledFn fn = get_encode_fn();
    if (fn == nullptr) return false;
    CUtensorMapSwizzle sw;
    switch (box_cols * 2) {
        case 32: sw = CU_TENSOR_MAP_SWIZZLE_32B; break;
        case 64: sw = CU_TENSOR_MAP_SWIZZLE_64B; break;
        case 128: sw = CU_TENSOR_MAP_SWIZZLE_128B; break;
        default: return false;
    }
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 row-major [rows, cols] -> map with a box of `box_rows` rows x 64 columns, 128-byte swizzle.
bool make_weight_map(CUtensorMap* tm, void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    return make_map_2d(tm, ptr, rows, cols, box_rows, 64);
}

}  // namespace
