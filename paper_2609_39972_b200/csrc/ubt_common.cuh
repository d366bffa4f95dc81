// Shared device helpers of the UBTree hot-path kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ubt {

constexpr unsigned FULL = 0xffffffffu;
constexpr float kLog2e = 1.4426950408889634f;

// ---------------------------------------------------------------- ordering keys
// Monotone map float -> uint32 (larger float <=> larger key); -0 and +0 share a key.
// NaN has no place in the order; the callers document NaN-free inputs.
__device__ __forceinline__ uint32_t f2key(float x) {
  uint32_t b = __float_as_uint(__fadd_rn(x, 0.0f));  // -0 + 0 = +0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key2f(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
// Largest float strictly below x in the numeric order (x finite or +inf; -0 and +0 are one value).
__device__ __forceinline__ float next_below(float x) {
  uint32_t k = f2key(x) - 1u;
  if (k == 0x7fffffffu) k = 0x7ffffffeu;  // the key of -0 is never produced; step over it
  return key2f(k);
}
// (value desc, index asc) as one descending 64-bit key.
__device__ __forceinline__ uint64_t make_key(float x, int idx) {
  return ((uint64_t)f2key(x) << 32) | (uint32_t)(~(uint32_t)idx);
}
__device__ __forceinline__ int key_idx(uint64_t k) { return (int)(~(uint32_t)k); }
__device__ __forceinline__ float key_val(uint64_t k) { return key2f((uint32_t)(k >> 32)); }

// ---------------------------------------------------------------- streaming loads
__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// One 16-byte fragment of a logits row as floats.
template <typename T> struct Frag;
template <> struct Frag<__nv_bfloat16> {
  static constexpr int N = 8;
  float x[8];
  __device__ __forceinline__ void unpack(const uint4& v) {
    x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
    x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
    x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xffff0000u);
    x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xffff0000u);
  }
};
template <> struct Frag<float> {
  static constexpr int N = 4;
  float x[4];
  __device__ __forceinline__ void unpack(const uint4& v) {
    x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
    x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
  }
};

__device__ __forceinline__ float load_elem(const __nv_bfloat16* p, int64_t i) {
  return __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(p)[i] << 16);
}
__device__ __forceinline__ float load_elem(const float* p, int64_t i) { return p[i]; }

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---------------------------------------------------------------- packed pairs of floats (one FFMA2 / FADD2 per pair)
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// ---------------------------------------------------------------- programmatic dependent launch
// A kernel launched with the programmatic-stream-serialization attribute may start while the kernel before
// it in the stream is still running, once every CTA of that kernel has called pdl_launch_dependents() (or
// exited); pdl_wait() blocks until the earlier kernel has completed and its writes are visible.  Both are
// no-ops for a kernel that was launched without the attribute / has no such successor.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------- warp / block reductions
__device__ __forceinline__ uint64_t warp_max_u64(uint64_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    uint64_t w = __shfl_xor_sync(FULL, v, o);
    v = w > v ? w : v;
  }
  return v;
}
__device__ __forceinline__ uint64_t warp_sum_u64(uint64_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
  return v;
}

// ---------------------------------------------------------------- checked array views
// With -DUBT_BOUNDS_CHECK every indexed access through a Span is range-checked; the first violation is
// recorded (site, index, limit) in a per-translation-unit device word and the access is redirected to
// element 0, so a wrong index is reported instead of faulting.  Without the flag a Span is a bare pointer.
#ifdef UBT_BOUNDS_CHECK
struct BoundsReport { unsigned int flag; int site; long long index; long long limit; };
static __device__ BoundsReport g_bounds_report;
static __device__ __noinline__ void bounds_violation(int site, long long i, long long n) {
  if (atomicCAS(&g_bounds_report.flag, 0u, 1u) == 0u) {
    g_bounds_report.site = site; g_bounds_report.index = i; g_bounds_report.limit = n;
  }
}
template <typename T> struct Span {
  T* p; long long n; int site;
  __host__ __device__ Span() : p(nullptr), n(0), site(0) {}
  __host__ __device__ Span(T* p_, long long n_, int site_) : p(p_), n(n_), site(site_) {}
  __device__ __forceinline__ T& operator[](long long i) const {
    if (i < 0 || i >= n) { bounds_violation(site, i, n); return p[0]; }
    return p[i];
  }
  __device__ __forceinline__ T* ptr(long long i, long long count) const {  // checked sub-range
    if (i < 0 || i + count > n) { bounds_violation(site, i, n); return p; }
    return p + i;
  }
};
#else
template <typename T> struct Span {
  T* p;
  __host__ __device__ Span() : p(nullptr) {}
  __host__ __device__ Span(T* p_, long long, int) : p(p_) {}
  __device__ __forceinline__ T& operator[](long long i) const { return p[i]; }
  __device__ __forceinline__ T* ptr(long long i, long long) const { return p + i; }
};
#endif

// How a flat range of rows*V elements is cut into per-CTA spans.
struct SpanPlan {
  int64_t span;  // elements per CTA (multiple of 256)
  int grid;      // CTAs
  int smax;      // partial slots per row: a row meets at most this many spans
};

}  // namespace ubt
