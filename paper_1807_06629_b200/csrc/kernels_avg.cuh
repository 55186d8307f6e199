// Node average over the stacked worker axis (Algorithm 1: y = (1/N) sum_i x_i)
// with the restart broadcast in the same pass, plus small store utilities.
// Every column is summed in worker order i = 0..N-1 in fp32 and divided by N
// once, so the result does not depend on the launch shape.
#pragma once
#include "prsgd_common.cuh"

namespace prsgd {

__device__ __forceinline__ void st_stream(float4* p, float4 v) { __stcs(p, v); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t a = __float_as_uint(lo), b = __float_as_uint(hi);
  a += 0x7FFFu + ((a >> 16) & 1u);
  b += 0x7FFFu + ((b >> 16) & 1u);
  return (a >> 16) | (b & 0xFFFF0000u);
}

template <int V> struct LaneVec;
template <> struct LaneVec<4> { using type = float4; };
template <> struct LaneVec<2> { using type = float2; };

__device__ __forceinline__ void acc_lane(float4& s, const float4& v) { s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w; }
__device__ __forceinline__ void acc_lane(float2& s, const float2& v) { s.x += v.x; s.y += v.y; }
__device__ __forceinline__ float4 div_lane(const float4& s, float n) {
  return make_float4(__fdiv_rn(s.x, n), __fdiv_rn(s.y, n), __fdiv_rn(s.z, n), __fdiv_rn(s.w, n));
}
__device__ __forceinline__ float2 div_lane(const float2& s, float n) { return make_float2(__fdiv_rn(s.x, n), __fdiv_rn(s.y, n)); }
__device__ __forceinline__ void st_shadow(uint16_t* row, int64_t c, const float4& y) {
  reinterpret_cast<uint2*>(row)[c] = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
}
__device__ __forceinline__ void st_shadow(uint16_t* row, int64_t c, const float2& y) {
  reinterpret_cast<uint32_t*>(row)[c] = pack_bf16x2(y.x, y.y);
}

// MODE 0: average + broadcast in place; MODE 1: average only, written to `out` (one row);
// MODE 2: plain sum of the rows (no division) written to `out`: the local part of an average whose
// rows are spread over several GPUs.
// One thread owns V consecutive columns (a 128-bit lane for V = 4, a 64-bit lane for V = 2); the tail
// m % V is done by scalar threads.  V = 2 doubles the number of blocks, which evens out the load of
// the SMs when a row is so short that 128-bit lanes give less than about two waves of blocks.
template <int MODE, bool SHADOW, int V = 4>
__global__ void __launch_bounds__(256) average_rows_kernel(float* __restrict__ P, int64_t N, int64_t m,
                                                           int64_t row_stride, float* __restrict__ out,
                                                           uint16_t* __restrict__ shadow,
                                                           const DeviceStatus* status = nullptr, float divisor = 0.f) {
  using Vec = typename LaneVec<V>::type;
  constexpr int U = 8;
  asm volatile("griddepcontrol.wait;" ::: "memory");   // no-op unless launched as a programmatic dependent
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // after the wait, like every kernel of the tensor-core path
  if (status != nullptr && status->error != 0u) return;   // a recorded expired wait: leave the store alone
  const int64_t colsV = m / V;
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const float fN = divisor > 0.f ? divisor : (float)N;      // (divisor 1: every row receives the row SUM)
  if (c < colsV) {
    Vec* base = reinterpret_cast<Vec*>(P) + c;
    const int64_t sV = row_stride / V;
    Vec s = Vec();
    int64_t i = 0;
    for (; i + U <= N; i += U) {
      Vec v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) v[u] = __ldcs(base + (i + u) * sV);
#pragma unroll
      for (int u = 0; u < U; ++u) acc_lane(s, v[u]);
    }
    for (; i < N; ++i) acc_lane(s, __ldcs(base + i * sV));
    const Vec y = MODE == 2 ? s : div_lane(s, fN);
    if (MODE == 0) {
#pragma unroll 8
      for (int64_t r = 0; r < N; ++r) __stcs(base + r * sV, y);
      if (SHADOW) {
        for (int64_t r = 0; r < N; ++r) st_shadow(shadow + r * row_stride, c, y);
      }
    } else {
      reinterpret_cast<Vec*>(out)[c] = y;
    }
  } else if (c < colsV + (m % V)) {
    const int64_t j = colsV * V + (c - colsV);
    float s = 0.f;
    for (int64_t i = 0; i < N; ++i) s += P[i * row_stride + j];
    float y = MODE == 2 ? s : __fdiv_rn(s, fN);
    if (MODE == 0) {
      for (int64_t r = 0; r < N; ++r) P[r * row_stride + j] = y;
      if (SHADOW) {
        for (int64_t r = 0; r < N; ++r) shadow[r * row_stride + j] = (uint16_t)(pack_bf16x2(y, 0.f) & 0xFFFFu);
      }
    } else {
      out[j] = y;
    }
  }
}

// Rows shorter than this many columns are averaged with 64-bit lanes (see average_rows_kernel).
constexpr int64_t kAvgNarrowLaneBelow = 8000000;

// every row <- src / divisor on columns [0, 4 * cols4) (and the bf16 shadow): the restart after an
// average whose sum was formed elsewhere (all-reduce over GPUs)
template <bool SHADOW>
__global__ void __launch_bounds__(256) assign_rows_kernel(float* __restrict__ P, uint16_t* __restrict__ shadow,
                                                          const float* __restrict__ src, float divisor, int64_t N,
                                                          int64_t cols4, int64_t stride4, const DeviceStatus* status) {
  if (status != nullptr && status->error != 0u) return;
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= cols4) return;
  const float4 s = reinterpret_cast<const float4*>(src)[c];
  const float4 y = make_float4(__fdiv_rn(s.x, divisor), __fdiv_rn(s.y, divisor), __fdiv_rn(s.z, divisor), __fdiv_rn(s.w, divisor));
  float4* base = reinterpret_cast<float4*>(P) + c;
  for (int64_t r = 0; r < N; ++r) st_stream(base + r * stride4, y);
  if (SHADOW) {
    const uint2 h = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
    uint2* sb = reinterpret_cast<uint2*>(shadow) + c;
    for (int64_t r = 0; r < N; ++r) sb[r * stride4] = h;
  }
}

// Finite check: counts the words of `P` (total4 float4 lanes, rows of row4 lanes) whose exponent field is
// all ones (NaN or +-infinity) and records the lowest row that holds one.  Reads only.
__global__ void __launch_bounds__(256) finite_check_kernel(const float* __restrict__ P, int64_t total4, int64_t row4,
                                                           DeviceStatus* status) {
  unsigned int bad = 0u, row = 0xFFFFFFFFu;
  for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < total4; c += (int64_t)gridDim.x * blockDim.x) {
    const uint4 v = __ldcs(reinterpret_cast<const uint4*>(P) + c);
    const unsigned int k = ((v.x & 0x7F800000u) == 0x7F800000u) + ((v.y & 0x7F800000u) == 0x7F800000u) +
                           ((v.z & 0x7F800000u) == 0x7F800000u) + ((v.w & 0x7F800000u) == 0x7F800000u);
    if (k != 0u) {
      bad += k;
      const unsigned int r = (unsigned int)(c / row4);
      row = r < row ? r : row;
    }
  }
  if (bad != 0u) {                       // rare: the atomics cost nothing on a healthy store
    const unsigned int old = atomicAdd(&status->nonfinite, bad);
    if (old + bad < old) atomicExch(&status->nonfinite, 0xFFFFFFFFu);   // saturate instead of wrapping
    atomicMin(&status->nonfinite_row, row);
  }
}

// device-resident iteration counter of a captured period: set before a replay, advanced at its end
__global__ void counter_set_kernel(int64_t* counter, int64_t value) { *counter = value; }
__global__ void counter_add_kernel(int64_t* counter, int64_t delta) {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  *counter += delta;
}

// rows 1..N-1 <- row 0 (every worker starts from the same point; Algorithm 1, input line)
__global__ void __launch_bounds__(256) broadcast_row0_kernel(float* __restrict__ P, int64_t N, int64_t cols4,
                                                             int64_t stride4) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= cols4) return;
  float4* base = reinterpret_cast<float4*>(P) + c;
  float4 v = base[0];
  for (int64_t r = 1; r < N; ++r) base[r * stride4] = v;
}

// shadow <- bf16(store), whole [N][m_pad] array
__global__ void __launch_bounds__(256) refresh_shadow_kernel(const float* __restrict__ P, uint16_t* __restrict__ S,
                                                             int64_t total4) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= total4) return;
  float4 v = reinterpret_cast<const float4*>(P)[c];
  reinterpret_cast<uint2*>(S)[c] = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
}

// Rows of the store (or of the momentum buffers) <-> rows in canonical order (W_1 row-major, b_1, W_2, ...
// without gaps).  A tile-major weight segment (see WTile) is permuted on the way; everything else is a copy.
// Grid (blocks, 2 L, rows): blockIdx.y = 2 (l - 1) for W_l, + 1 for b_l.
struct CanonArgs {
  int L;
  int64_t w_off[PRSGD_MAX_LAYERS], b_off[PRSGD_MAX_LAYERS];       // offsets inside a store row
  int64_t w_pos[PRSGD_MAX_LAYERS], b_pos[PRSGD_MAX_LAYERS];       // offsets inside a canonical row
  int d_out[PRSGD_MAX_LAYERS];
  WTile wt[PRSGD_MAX_LAYERS];
};

__global__ void __launch_bounds__(256) canonical_copy_kernel(float* __restrict__ store, int64_t store_stride,
                                                             float* __restrict__ lin, int64_t lin_stride,
                                                             const CanonArgs a, int to_store) {
  const int l = blockIdx.y >> 1, is_bias = blockIdx.y & 1;
  float* srow = store + (int64_t)blockIdx.z * store_stride + (is_bias ? a.b_off[l] : a.w_off[l]);
  float* lrow = lin + (int64_t)blockIdx.z * lin_stride + (is_bias ? a.b_pos[l] : a.w_pos[l]);
  const int d_in = a.wt[l].d_in;
  const int64_t len = is_bias ? (int64_t)a.d_out[l] : (int64_t)a.d_out[l] * d_in;
  for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < len; j += (int64_t)gridDim.x * blockDim.x) {
    const int64_t o = (is_bias || !a.wt[l].tiled) ? j : wtile_offset(a.wt[l], (int)(j / d_in), (int)(j % d_in));
    if (to_store) srow[o] = lrow[j];
    else lrow[j] = srow[o];
  }
}

}  // namespace prsgd
