// Device helpers shared by the GTO kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace gto {

constexpr int kWarp = 32;
constexpr unsigned kFull = 0xffffffffu;

// bits of the device status word
constexpr int kStatusNonFinite = 1;
constexpr int kStatusBadIndex = 4;  // an index read from a caller's table was out of range

constexpr float kLog2e = 1.4426950408889634f;
constexpr double kLn2 = 0.6931471805599453094;

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 16-byte streaming load: read-only path, no L1 allocation (every byte is used once).
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void st_stream16(void* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}

// Logit element types.  A "vector" is 16 bytes: 8 bf16 or 4 fp32 values.
struct Bf16 {
  static constexpr int kPerVec = 8;
  static constexpr int kBytes = 2;
  static constexpr uint32_t kNegInfWord = 0xff80ff80u;
  using Storage = uint16_t;
  static constexpr Storage kNegInfElem = 0xff80u;
  // stored bits of element e of a vector
  __device__ static __forceinline__ Storage element(const uint4& v, int e) {
    const uint32_t w = e < 4 ? (e < 2 ? v.x : v.y) : (e < 6 ? v.z : v.w);
    return static_cast<Storage>(e & 1 ? w >> 16 : w & 0xffffu);
  }
  __device__ static __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
    f[0] = __uint_as_float(v.x << 16);
    f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16);
    f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16);
    f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16);
    f[7] = __uint_as_float(v.w & 0xffff0000u);
  }
  __device__ static __forceinline__ uint4 pack(const float (&f)[8]) {
    uint4 v;
    __nv_bfloat162 a = __floats2bfloat162_rn(f[0], f[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(f[2], f[3]);
    __nv_bfloat162 c = __floats2bfloat162_rn(f[4], f[5]);
    __nv_bfloat162 d = __floats2bfloat162_rn(f[6], f[7]);
    v.x = *reinterpret_cast<uint32_t*>(&a);
    v.y = *reinterpret_cast<uint32_t*>(&b);
    v.z = *reinterpret_cast<uint32_t*>(&c);
    v.w = *reinterpret_cast<uint32_t*>(&d);
    return v;
  }
  __device__ static __forceinline__ float load1(const void* base, size_t idx) {
    return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(base)[idx]);
  }
  // Running maximum kept as two packed bf16 lanes (4 instructions per 8 logits).
  using MaxAcc = uint32_t;
  __device__ static __forceinline__ MaxAcc max_init() { return kNegInfWord; }
  __device__ static __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
  }
  __device__ static __forceinline__ void max_update(MaxAcc& acc, const uint4& v) {
    acc = max2(acc, max2(max2(v.x, v.y), max2(v.z, v.w)));
  }
  __device__ static __forceinline__ float max_value(MaxAcc acc) {
    return fmaxf(__uint_as_float(acc << 16), __uint_as_float(acc & 0xffff0000u));
  }
};

struct F16 {
  static constexpr int kPerVec = 8;
  static constexpr int kBytes = 2;
  static constexpr uint32_t kNegInfWord = 0xfc00fc00u;
  using Storage = uint16_t;
  static constexpr Storage kNegInfElem = 0xfc00u;
  __device__ static __forceinline__ Storage element(const uint4& v, int e) {
    const uint32_t w = e < 4 ? (e < 2 ? v.x : v.y) : (e < 6 ? v.z : v.w);
    return static_cast<Storage>(e & 1 ? w >> 16 : w & 0xffffu);
  }
  __device__ static __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float2 p = __half22float2(*reinterpret_cast<const __half2*>(&w[q]));
      f[2 * q] = p.x;
      f[2 * q + 1] = p.y;
    }
  }
  __device__ static __forceinline__ uint4 pack(const float (&f)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const __half2 h = __floats2half2_rn(f[2 * q], f[2 * q + 1]);
      w[q] = *reinterpret_cast<const uint32_t*>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
  __device__ static __forceinline__ float load1(const void* base, size_t idx) {
    return __half2float(reinterpret_cast<const __half*>(base)[idx]);
  }
  // Running maximum kept as two packed fp16 lanes.
  using MaxAcc = uint32_t;
  __device__ static __forceinline__ MaxAcc max_init() { return kNegInfWord; }
  __device__ static __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
  }
  __device__ static __forceinline__ void max_update(MaxAcc& acc, const uint4& v) {
    acc = max2(acc, max2(max2(v.x, v.y), max2(v.z, v.w)));
  }
  __device__ static __forceinline__ float max_value(MaxAcc acc) {
    const float2 p = __half22float2(*reinterpret_cast<const __half2*>(&acc));
    return fmaxf(p.x, p.y);
  }
};

struct F32 {
  static constexpr int kPerVec = 4;
  static constexpr int kBytes = 4;
  static constexpr uint32_t kNegInfWord = 0xff800000u;
  using Storage = uint32_t;
  static constexpr Storage kNegInfElem = 0xff800000u;
  __device__ static __forceinline__ Storage element(const uint4& v, int e) {
    return e < 2 ? (e == 0 ? v.x : v.y) : (e == 2 ? v.z : v.w);
  }
  __device__ static __forceinline__ void unpack(const uint4& v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x);
    f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z);
    f[3] = __uint_as_float(v.w);
  }
  __device__ static __forceinline__ uint4 pack(const float (&f)[4]) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                      __float_as_uint(f[3]));
  }
  __device__ static __forceinline__ float load1(const void* base, size_t idx) {
    return reinterpret_cast<const float*>(base)[idx];
  }
  using MaxAcc = float;
  __device__ static __forceinline__ MaxAcc max_init() { return -INFINITY; }
  __device__ static __forceinline__ void max_update(MaxAcc& acc, const uint4& v) {
    acc = fmaxf(fmaxf(acc, fmaxf(__uint_as_float(v.x), __uint_as_float(v.y))),
                fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
  }
  __device__ static __forceinline__ float max_value(MaxAcc acc) { return acc; }
};

// Total order on (value, id): larger key = better candidate = (value desc, id asc).
__device__ __forceinline__ uint32_t orderable(float z) {
  uint32_t u = __float_as_uint(z + 0.0f);  // -0 -> +0
  return u ^ ((u >> 31) ? 0xffffffffu : 0x80000000u);
}
__device__ __forceinline__ uint64_t make_key(float z, int id) {
  return (static_cast<uint64_t>(orderable(z)) << 32) | (0xffffffffu - static_cast<uint32_t>(id));
}
__device__ __forceinline__ int key_id(uint64_t key) {
  return static_cast<int>(0xffffffffu - static_cast<uint32_t>(key));
}
// Inverse of orderable().
__device__ __forceinline__ float from_orderable(uint32_t o) {
  return __uint_as_float(o ^ ((o >> 31) ? 0x80000000u : 0xffffffffu));
}
__device__ __forceinline__ float key_value(uint64_t key) {
  return from_orderable(static_cast<uint32_t>(key >> 32));
}

__device__ __forceinline__ uint64_t warp_max_u64(uint64_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    uint64_t w = __shfl_xor_sync(kFull, v, o);
    v = w > v ? w : v;
  }
  return v;
}

__device__ __forceinline__ float warp_max_f32(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
  return v;
}

__device__ __forceinline__ float warp_sum_f32(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}

// Context row r of a tree -> row offset inside the tree's block of the logits tensor.
// The draft tensor [.,.,D,k,V] keeps k-1 unused rows between the root and row 1.
__device__ __forceinline__ int64_t tensor_row(int tree, int r, int R, int pad) {
  return static_cast<int64_t>(tree) * (R + pad) + r + (r > 0 ? pad : 0);
}

}  // namespace gto
