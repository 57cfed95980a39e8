// Storage formats of an expert row and their decoding, shared by the streaming expert-FFN kernel and the token kernel.
#ifndef APEX_FFN_ROWS_CUH
#define APEX_FFN_ROWS_CUH

#include <cuda_fp16.h>

#include <cstdint>

namespace apex {

__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

// Storage formats of an expert row (FfnParams::fmt)
constexpr int kFmtBf16 = 0;   // bf16
constexpr int kFmtE4m3 = 1;   // e4m3 codes, one fp32 scale per vector of the row
constexpr int kFmtMxfp4 = 2;  // e2m1 codes, one power-of-two scale (a biased exponent byte) per 32 elements

__host__ __device__ constexpr uint32_t fmt_vec_bytes(int fmt, int d) { return fmt == kFmtMxfp4 ? d / 2 : (fmt == kFmtE4m3 ? d : 2 * d); }
__host__ __device__ constexpr uint32_t fmt_entry_bytes(int fmt, int d) {
  return fmt == kFmtMxfp4 ? ((3u * (d / 2) + 3u * (d / 32) + 15u) & ~15u) : (fmt == kFmtE4m3 ? 3u * d + 16u : 6u * d);
}

// Eight consecutive weights of a vector as fp32: bf16 (16 bytes), e4m3 (8 bytes) or e2m1 (4 bytes); scales are
// applied by the caller.
template <int FMT>
__device__ __forceinline__ void load8(const uint8_t* row, int idx8, float (&w)[8]) {
  if (FMT == kFmtMxfp4) {
    const uint32_t v = reinterpret_cast<const uint32_t*>(row)[idx8];
    uint32_t h2[4];
    asm("{\n.reg .b8 b0, b1, b2, b3;\n"
        "mov.b32 {b0, b1, b2, b3}, %4;\n"
        "cvt.rn.f16x2.e2m1x2 %0, b0;\n"
        "cvt.rn.f16x2.e2m1x2 %1, b1;\n"
        "cvt.rn.f16x2.e2m1x2 %2, b2;\n"
        "cvt.rn.f16x2.e2m1x2 %3, b3;\n}"
        : "=r"(h2[0]), "=r"(h2[1]), "=r"(h2[2]), "=r"(h2[3])
        : "r"(v));
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h2[i]));
      w[2 * i] = f.x;
      w[2 * i + 1] = f.y;
    }
  } else if (FMT == kFmtE4m3) {
    const uint2 v = reinterpret_cast<const uint2*>(row)[idx8];
    uint32_t h2[4];
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2[0]) : "h"((unsigned short)(v.x & 0xffffu)));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2[1]) : "h"((unsigned short)(v.x >> 16)));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2[2]) : "h"((unsigned short)(v.y & 0xffffu)));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2[3]) : "h"((unsigned short)(v.y >> 16)));
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h2[i]));
      w[2 * i] = f.x;
      w[2 * i + 1] = f.y;
    }
  } else {
    const uint4 v = reinterpret_cast<const uint4*>(row)[idx8];
    w[0] = bf16lo(v.x); w[1] = bf16hi(v.x); w[2] = bf16lo(v.y); w[3] = bf16hi(v.y);
    w[4] = bf16lo(v.z); w[5] = bf16hi(v.z); w[6] = bf16lo(v.w); w[7] = bf16hi(v.w);
  }
}
// scale of the 32-element block that holds elements 8*idx8 .. 8*idx8+7 (block-scaled format only)
__device__ __forceinline__ float block_scale(const uint8_t* scales, int idx8) {
  return __uint_as_float((uint32_t)scales[idx8 >> 2] << 23);
}

}  // namespace apex

#endif  // APEX_FFN_ROWS_CUH
