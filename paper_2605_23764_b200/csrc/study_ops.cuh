// Row-tile bodies of the two element-wise operators of the scheduling microbenchmarks (Section 6): SwiGLU on rows of
// x[M][2C] (gate | up halves) and Add of two [M][C] tensors, bf16, 16 bytes per thread and step.  Shared by the
// fixed-schedule kernels (study.cu) and the task-descriptor runtime (taskflow.cu).
#pragma once

#include <cuda_bf16.h>

#include "common.cuh"

namespace moe {

constexpr int STUDY_THREADS = 256;

__device__ __forceinline__ uint4 ld_cg16(const void* p) {
  uint4 v;
  asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint4 ld_nc16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ float silu_mul(float g, float u) { return g * __fdividef(1.0f, 1.0f + __expf(-g)) * u; }
__device__ __forceinline__ uint32_t swiglu2(uint32_t g, uint32_t u) {
  return pack_bf16x2(silu_mul(bf16lo(g), bf16lo(u)), silu_mul(bf16hi(g), bf16hi(u)));
}
__device__ __forceinline__ uint32_t add2(uint32_t a, uint32_t b) {
  return pack_bf16x2(bf16lo(a) + bf16lo(b), bf16hi(a) + bf16hi(b));
}

// 16-byte vectors per thread in flight per operand: the one-operator kernels run four blocks per SM, the
// persistent workers two with twice the vectors each, so both keep the same number of bytes in flight per SM
constexpr int SERIAL_UNROLL = 4, WORKER_UNROLL = 2;

// SwiGLU of rows [r0, r1): s[m][c] = silu(x[m][c]) * x[m][C + c]; 8 columns per vector.  Byte offsets from
// the tile's first row stay in 32 bits (a tile is far smaller than 4 GB).
// COHERENT: x may have been written earlier in the same launch by another SM (read it at L2, not through the
// non-coherent path)
template <int STUDY_UNROLL, bool COHERENT = false>
__device__ __forceinline__ void swiglu_tile(const uint16_t* __restrict__ x, uint16_t* __restrict__ s, int C, int r0, int r1) {
  const uint32_t nvec = C >> 3, total = (r1 - r0) * nvec;
  const char* xb = reinterpret_cast<const char*>(x + (size_t)r0 * 2 * C);
  char* sb = reinterpret_cast<char*>(s + (size_t)r0 * C);
#pragma unroll 1
  for (uint32_t base = threadIdx.x; base < total; base += STUDY_UNROLL * STUDY_THREADS) {
    uint4 g[STUDY_UNROLL], u[STUDY_UNROLL];
#pragma unroll
    for (int j = 0; j < STUDY_UNROLL; ++j) {
      const uint32_t i = base + j * STUDY_THREADS;
      if (i < total) {
        const uint32_t off = (i + (i / nvec) * nvec) * 16u;   // row m, vector v of the gate half: (m * 2 nvec + v) * 16
        g[j] = COHERENT ? ld_cg16(xb + off) : ld_nc16(xb + off);
        u[j] = COHERENT ? ld_cg16(xb + off + nvec * 16u) : ld_nc16(xb + off + nvec * 16u);
      }
    }
#pragma unroll
    for (int j = 0; j < STUDY_UNROLL; ++j) {
      const uint32_t i = base + j * STUDY_THREADS;
      if (i < total) {
        uint4 o;
        o.x = swiglu2(g[j].x, u[j].x); o.y = swiglu2(g[j].y, u[j].y);
        o.z = swiglu2(g[j].z, u[j].z); o.w = swiglu2(g[j].w, u[j].w);
        *reinterpret_cast<uint4*>(sb + i * 16u) = o;
      }
    }
  }
}
// Add of rows [r0, r1): z = s + r.  s was written earlier (possibly in this launch, by another SM): read at L2.
template <int STUDY_UNROLL, bool COHERENT = false>
__device__ __forceinline__ void add_tile(const uint16_t* s, const uint16_t* __restrict__ r, uint16_t* __restrict__ z, int C,
                                         int r0, int r1) {
  const uint32_t total = (r1 - r0) * (C >> 3);
  const char* sb = reinterpret_cast<const char*>(s + (size_t)r0 * C);
  const char* rb = reinterpret_cast<const char*>(r + (size_t)r0 * C);
  char* zb = reinterpret_cast<char*>(z + (size_t)r0 * C);
#pragma unroll 1
  for (uint32_t base = threadIdx.x; base < total; base += STUDY_UNROLL * STUDY_THREADS) {
    uint4 a[STUDY_UNROLL], b[STUDY_UNROLL];
#pragma unroll
    for (int j = 0; j < STUDY_UNROLL; ++j) {
      const uint32_t i = base + j * STUDY_THREADS;
      if (i < total) {
        a[j] = ld_cg16(sb + i * 16u);
        b[j] = COHERENT ? ld_cg16(rb + i * 16u) : ld_nc16(rb + i * 16u);
      }
    }
#pragma unroll
    for (int j = 0; j < STUDY_UNROLL; ++j) {
      const uint32_t i = base + j * STUDY_THREADS;
      if (i < total) {
        uint4 o;
        o.x = add2(a[j].x, b[j].x); o.y = add2(a[j].y, b[j].y); o.z = add2(a[j].z, b[j].z); o.w = add2(a[j].w, b[j].w);
        *reinterpret_cast<uint4*>(zb + i * 16u) = o;
      }
    }
  }
}

}  // namespace moe
