// Element arithmetic shared by the boxing kernels of this library (device code only): the fp32
// lanes of a vector, the fixed-order combine, the streaming load.
#pragma once

#include <cuda_bf16.h>

#include <cstdint>

namespace sbp {

enum BoxOp : int { OP_COPY = 0, OP_SUM_F32, OP_SUM_BF16, OP_MAX_F32, OP_MAX_BF16 };

// ------------------------------------------------------------------ element arithmetic

// fp32 lanes carried by one vector of type V
template <typename V>
struct AccF32 {
  static constexpr int N = sizeof(V) / 4;
  float v[N];
  __device__ void load(const V& x) {
    const float* f = reinterpret_cast<const float*>(&x);
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = f[i];
  }
  __device__ V store() const {
    V out;
    float* f = reinterpret_cast<float*>(&out);
#pragma unroll
    for (int i = 0; i < N; ++i) f[i] = v[i];
    return out;
  }
};

template <typename V>
struct AccBF16 {
  static constexpr int N = sizeof(V) / 2;
  float v[N];
  __device__ void load(const V& x) {
    const __nv_bfloat16* h = reinterpret_cast<const __nv_bfloat16*>(&x);
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = __bfloat162float(h[i]);
  }
  __device__ V store() const {
    V out;
    __nv_bfloat16* h = reinterpret_cast<__nv_bfloat16*>(&out);
#pragma unroll
    for (int i = 0; i < N; ++i) h[i] = __float2bfloat16_rn(v[i]);   // the single rounding
    return out;
  }
};

template <int OP, typename V>
struct Lanes {
  using type = AccF32<V>;
};
template <typename V>
struct Lanes<OP_SUM_BF16, V> {
  using type = AccBF16<V>;
};
template <typename V>
struct Lanes<OP_MAX_BF16, V> {
  using type = AccBF16<V>;
};

template <int OP, typename L>
__device__ __forceinline__ void combine(L& acc, const L& x) {
#pragma unroll
  for (int i = 0; i < L::N; ++i) {
    if (OP == OP_SUM_F32 || OP == OP_SUM_BF16)
      acc.v[i] = __fadd_rn(acc.v[i], x.v[i]);          // plain IEEE add, never contracted
    else
      acc.v[i] = (x.v[i] > acc.v[i]) ? x.v[i] : acc.v[i];   // first wins on ties
  }
}

template <typename V>
__device__ __forceinline__ V ld_stream(const V* p) {
  return *p;
}
template <>
__device__ __forceinline__ uint4 ld_stream<uint4>(const uint4* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

// Stores of results that this kernel never reads again: the 16-byte form is marked evict-first
// so that the output stream does not push the inputs still to be read out of L2.
template <typename V>
__device__ __forceinline__ void st_stream(V* p, const V& v) {
  *p = v;
}
template <>
__device__ __forceinline__ void st_stream<uint4>(uint4* p, const uint4& v) {
  __stcs(p, v);
}

}  // namespace sbp
