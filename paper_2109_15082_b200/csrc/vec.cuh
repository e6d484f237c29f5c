// 16-byte vector access for float32 / bfloat16 tensors and packed 8-bit codes.
#pragma once
#include "mrem_common.cuh"

namespace mrem {

template <typename T, int V>
__device__ __forceinline__ void load_vec(const T* p, float* v) {
  if constexpr (V == 1) {
    v[0] = to_f<T>(p[0]);
  } else if constexpr (sizeof(T) == 4) {
    static_assert(V == 4, "float vectors hold 4 values");
    const float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  } else if constexpr (V == 2) {
    const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p));
    v[0] = f.x; v[1] = f.y;
  } else if constexpr (V == 4) {
    const uint2 t = *reinterpret_cast<const uint2*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&t);
    const float2 f0 = __bfloat1622float2(h[0]), f1 = __bfloat1622float2(h[1]);
    v[0] = f0.x; v[1] = f0.y; v[2] = f1.x; v[3] = f1.y;
  } else {
    static_assert(V == 8, "bfloat16 vectors hold 2, 4 or 8 values");
    const uint4 t = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&t);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(h[i]);
      v[2 * i] = f.x;
      v[2 * i + 1] = f.y;
    }
  }
}

// The same load in two halves: the raw words first (V * sizeof(T) bytes, at most 16, in RAW_WORDS 32-bit
// registers), widened to float later, so that several loads can be in flight on few registers.
template <typename T, int V> struct RawWords { static constexpr int N = (V * (int)sizeof(T) + 3) / 4; };
template <typename T, int V>
__device__ __forceinline__ void load_raw(const T* p, uint32_t* w) {
  if constexpr (V * sizeof(T) == 16) {
    const uint4 t = *reinterpret_cast<const uint4*>(p);
    w[0] = t.x; w[1] = t.y; w[2] = t.z; w[3] = t.w;
  } else if constexpr (V * sizeof(T) == 8) {
    const uint2 t = *reinterpret_cast<const uint2*>(p);
    w[0] = t.x; w[1] = t.y;
  } else if constexpr (V * sizeof(T) == 4) {
    w[0] = *reinterpret_cast<const uint32_t*>(p);
  } else {
    static_assert(V == 1 && sizeof(T) == 2, "raw loads cover 2, 4, 8 and 16 bytes");
    w[0] = *reinterpret_cast<const unsigned short*>(p);
  }
}
template <typename T, int V>
__device__ __forceinline__ void widen_raw(const uint32_t* w, float* v) {
  if constexpr (sizeof(T) == 4) {
#pragma unroll
    for (int i = 0; i < V; ++i) v[i] = __uint_as_float(w[i]);
  } else if constexpr (V == 1) {
    v[0] = __uint_as_float(w[0] << 16);
  } else {
#pragma unroll
    for (int i = 0; i < V / 2; ++i) {
      const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
      v[2 * i] = f.x;
      v[2 * i + 1] = f.y;
    }
  }
}

template <typename T, int V>
__device__ __forceinline__ void store_vec(T* p, const float* v) {
  if constexpr (V == 1) {
    p[0] = from_f<T>(v[0]);
  } else if constexpr (sizeof(T) == 4) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  } else {
    uint4 t;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&t);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    *reinterpret_cast<uint4*>(p) = t;
  }
}

// V codes given as the bit patterns of rne_magic (low byte = the 8-bit code) packed into V bytes.
template <int V>
__device__ __forceinline__ void store_code_bytes(int8_t* p, const uint32_t* b) {
  if constexpr (V == 1) {
    p[0] = (int8_t)(b[0] & 0xff);
  } else if constexpr (V == 4) {
    *reinterpret_cast<uint32_t*>(p) = pack_low_bytes(b[0], b[1], b[2], b[3]);
  } else {
    static_assert(V == 8, "code vectors hold 1, 4 or 8 values");
    *reinterpret_cast<uint2*>(p) = make_uint2(pack_low_bytes(b[0], b[1], b[2], b[3]), pack_low_bytes(b[4], b[5], b[6], b[7]));
  }
}

// V integer codes (each fits 8 bits, signed or unsigned) packed into V bytes.
template <int V>
__device__ __forceinline__ void store_codes(int8_t* p, const int* q) {
  if constexpr (V == 1) {
    p[0] = (int8_t)q[0];
  } else if constexpr (V == 4) {
    uint32_t w = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) w |= (uint32_t)(q[i] & 0xff) << (8 * i);
    *reinterpret_cast<uint32_t*>(p) = w;
  } else {
    uint32_t w0 = 0, w1 = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      w0 |= (uint32_t)(q[i] & 0xff) << (8 * i);
      w1 |= (uint32_t)(q[i + 4] & 0xff) << (8 * i);
    }
    *reinterpret_cast<uint2*>(p) = make_uint2(w0, w1);
  }
}

}  // namespace mrem
