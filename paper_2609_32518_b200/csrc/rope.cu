// RoPE coefficient table and the fused RoPE + KV-ring append (HBM-bound kernels).
#include <cuda_bf16.h>

#include "common.h"

namespace unstep {

// --------------------------------------------------------------------------
// Table: one thread per (token, pair).  Angle and trig in double, one rounding.
// --------------------------------------------------------------------------
struct TableParams {
  int32_t start_frame, grid_h, grid_w, L;
  int32_t pairs_t, pairs_h;  // pairs_w = 64 - pairs_t - pairs_h
  int32_t band_t, band_h, band_w;
  double base;
  int* status;       // status word and extent (floats) of each output, for checking builds
  int64_t extent;
};

// cos and sin of position * omega in double, rounded once.
__device__ __forceinline__ float2 table_entry(double omega, int pos) {
  double sn, cs;
  sincos(static_cast<double>(pos) * omega, &sn, &cs);
  return make_float2(static_cast<float>(cs), static_cast<float>(sn));
}

// One block per (frame, token row).  The table is separable: a token's 64 coefficients are
// 22 that depend on its frame only, 21 on its row only and 21 on its column only.  The block
// evaluates those (22 + 21 + 21 * grid_w double-precision values) once into shared memory and
// then writes its grid_w * 64 entries of cos and sin with coalesced stores (64 columns per pass).  Evaluating every
// entry on its own costs 64 double pow/sincos per token instead of about 22.
__global__ void __launch_bounds__(1024) rope_table_kernel(TableParams p, float* __restrict__ cos_out,
                                                         float* __restrict__ sin_out) {
  constexpr int kColsPerPass = 64;
  __shared__ float2 band[kPairs + kColsPerPass * kPairs];   // frame/row part, then [column][pair]
  __shared__ double omega[kPairs];                          // base^(-2i/d_band) of the 64 pairs
  const int r = blockIdx.x, f = blockIdx.y;
  const int pairs_w = kPairs - p.pairs_t - p.pairs_h;
  const int n_fixed = p.pairs_t + p.pairs_h;
  if (threadIdx.x < kPairs) {
    const int j = threadIdx.x;
    const int i = j < p.pairs_t ? j : (j < n_fixed ? j - p.pairs_t : j - n_fixed);
    const int d = j < p.pairs_t ? p.band_t : (j < n_fixed ? p.band_h : p.band_w);
    omega[j] = pow(p.base, -(2.0 * static_cast<double>(i)) / static_cast<double>(d));
  }
  __syncthreads();
  const int64_t row_base = (static_cast<int64_t>(f) * p.grid_h + r) * p.grid_w * kPairs;
  for (int c0 = 0; c0 < p.grid_w; c0 += kColsPerPass) {
    const int cols = min(kColsPerPass, p.grid_w - c0);
    const int n_eval = n_fixed + cols * pairs_w;
    for (int e = threadIdx.x; e < n_eval; e += blockDim.x) {
      if (e < p.pairs_t) {
        band[e] = table_entry(omega[e], p.start_frame + f);
      } else if (e < n_fixed) {
        band[e] = table_entry(omega[e], r);
      } else {
        const int c = (e - n_fixed) / pairs_w, i = (e - n_fixed) - c * pairs_w;
        band[e] = table_entry(omega[n_fixed + i], c0 + c);
      }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < cols * kPairs; idx += blockDim.x) {
      const int c = idx >> 6, j = idx & 63;
      const float2 v = j < n_fixed ? band[j] : band[n_fixed + c * pairs_w + (j - n_fixed)];
      UNSTEP_STORE(cos_out, row_base + c0 * kPairs + idx, p.extent, v.x, p.status);
      UNSTEP_STORE(sin_out, row_base + c0 * kPairs + idx, p.extent, v.y, p.status);
    }
    __syncthreads();
  }
}

// --------------------------------------------------------------------------
// Append: one thread per 16-byte vector (8 bf16 = 4 pairs) of the same position in
// q, k and v.  Inputs are read once (streaming loads); outputs are re-read by the
// attention kernel right after, so they are left to the default cache policy.
// --------------------------------------------------------------------------
struct AppendParams {
  int32_t L, T, C, S, vec_per_token;  // C ring slots behind S sink slots; vec_per_token = Hn * 16
  int64_t vec_per_stream;          // L * Hn * 16
  int64_t ring_vec_per_stream;     // (S + C) * T * Hn * 16
  int64_t table_stream_stride;     // elements
  int32_t start[kMaxStreamsPerLaunch];  // start_frame[b]
  int* status;                     // status word and extents (16-byte vectors) of q_out and of the cache
  int64_t extent_act, extent_cache;     // of this launch's streams, for checking builds
};

__device__ __forceinline__ uint32_t rotate_pair(uint32_t w, float c, float s) {
  const float xe = __uint_as_float(w << 16);
  const float xo = __uint_as_float(w & 0xFFFF0000u);
  // four products, one difference, one sum, each rounded to float32: no contraction
  const float ye = __fsub_rn(__fmul_rn(xe, c), __fmul_rn(xo, s));
  const float yo = __fadd_rn(__fmul_rn(xe, s), __fmul_rn(xo, c));
  const __nv_bfloat162 y = __floats2bfloat162_rn(ye, yo);
  return *reinterpret_cast<const uint32_t*>(&y);
}

__device__ __forceinline__ uint4 rotate_vec(uint4 x, float4 c, float4 s) {
  uint4 y;
  y.x = rotate_pair(x.x, c.x, s.x);
  y.y = rotate_pair(x.y, c.y, s.y);
  y.z = rotate_pair(x.z, c.z, s.z);
  y.w = rotate_pair(x.w, c.w, s.w);
  return y;
}

__global__ void __launch_bounds__(256)
rope_kv_append_kernel(AppendParams p, const uint4* q_in, const uint4* __restrict__ k_in,
                      const uint4* __restrict__ v_in, const float4* __restrict__ cos_t,
                      const float4* __restrict__ sin_t, uint4* q_out,
                      uint4* __restrict__ ring_k, uint4* __restrict__ ring_v) {
  const int b = blockIdx.y;
  const int64_t v = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (v >= p.vec_per_stream) return;
  const int n = static_cast<int>(v / p.vec_per_token);
  const int rem = static_cast<int>(v - static_cast<int64_t>(n) * p.vec_per_token);
  const int f = n / p.T, t = n - f * p.T;
  // frames below S live in the sink prefix for good, later frames in the ring behind it
  const int frame = p.start[b] + f;
  const int slot = frame < p.S ? frame : p.S + (frame - p.S) % p.C;

  const int64_t in_idx = static_cast<int64_t>(b) * p.vec_per_stream + v;
  const uint4 xq = __ldcs(q_in + in_idx);
  const uint4 xk = __ldcs(k_in + in_idx);
  const uint4 xv = __ldcs(v_in + in_idx);
  const int64_t tab = (static_cast<int64_t>(b) * p.table_stream_stride >> 2) +
                      static_cast<int64_t>(n) * (kPairs / 4) + (rem & 15);
  const float4 c = __ldg(cos_t + tab);
  const float4 s = __ldg(sin_t + tab);

  const int64_t ring_idx = static_cast<int64_t>(b) * p.ring_vec_per_stream +
                           (static_cast<int64_t>(slot) * p.T + t) * p.vec_per_token + rem;
  UNSTEP_STORE(q_out, in_idx, p.extent_act, rotate_vec(xq, c, s), p.status);
  UNSTEP_STORE(ring_k, ring_idx, p.extent_cache, rotate_vec(xk, c, s), p.status);
  UNSTEP_STORE(ring_v, ring_idx, p.extent_cache, xv, p.status);
}

// --------------------------------------------------------------------------
// RMSNorm of q and k fused in front of the rotation.  The norm runs over the whole token
// vector (all heads).  The squares of a token's q and k are summed in double.  Each square is
// exact; the additions round at 2^-53 relative, so a sum taken in another order than the
// reference's can differ from it in the last bits of the double (and not at all unless the
// squares of one token span more than about 2^26 in magnitude), far below the rounding of the
// mean to float32 that follows: the float32 mean, and with it every output bit, does not depend
// on the order except in a near-tie of that rounding.  Then the token is normalised (float32:
// sqrt, reciprocal and two products, each rounded once), rounded to bf16 as the unfused pipeline
// would, rotated and stored.  Two kernels: a thread block per token that keeps the token in
// registers between the sum and the store (up to 64 heads), and a warp per token that reads q
// and k a second time from L1/L2 (wider tokens, which would not fit the registers of a block).
// --------------------------------------------------------------------------

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
  return x;
}
// Sum of the squares of the 8 bf16 of a vector, in double.  A bf16 square has 16 significant
// bits, so each fused multiply-add adds an exact square and rounds once, like the additions of
// the reference's double-precision sum.
__device__ __forceinline__ double squares(uint4 x, double acc) {
  double s0 = acc, s1 = 0.0;
  const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const double lo = static_cast<double>(__uint_as_float(w[i] << 16));
    const double hi = static_cast<double>(__uint_as_float(w[i] & 0xFFFF0000u));
    s0 = fma(lo, lo, s0);
    s1 = fma(hi, hi, s1);
  }
  return s0 + s1;
}
// y = bf16(fl32(fl32(x * r) * g)) for the 8 elements of a vector
__device__ __forceinline__ uint4 normalise_vec(uint4 x, float r, float4 g0, float4 g1) {
  const uint32_t w[4] = {x.x, x.y, x.z, x.w};
  const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
  uint32_t y[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float lo = __fmul_rn(__fmul_rn(__uint_as_float(w[i] << 16), r), g[2 * i]);
    const float hi = __fmul_rn(__fmul_rn(__uint_as_float(w[i] & 0xFFFF0000u), r), g[2 * i + 1]);
    const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    y[i] = *reinterpret_cast<const uint32_t*>(&b);
  }
  return make_uint4(y[0], y[1], y[2], y[3]);
}

__global__ void __launch_bounds__(256)
rmsnorm_rope_kv_append_kernel(AppendParams p, float eps, const uint4* q_in, const uint4* __restrict__ k_in,
                              const uint4* __restrict__ v_in, const float4* __restrict__ gain_q,
                              const float4* __restrict__ gain_k, const float4* __restrict__ cos_t,
                              const float4* __restrict__ sin_t, uint4* q_out, uint4* __restrict__ ring_k,
                              uint4* __restrict__ ring_v) {
  const int b = blockIdx.y;
  const int lane = threadIdx.x & 31;
  const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // token of this warp
  if (n >= p.L) return;
  const int f = n / p.T, t = n - f * p.T;
  const int frame = p.start[b] + f;
  const int slot = frame < p.S ? frame : p.S + (frame - p.S) % p.C;
  const int64_t in_base = static_cast<int64_t>(b) * p.vec_per_stream + static_cast<int64_t>(n) * p.vec_per_token;
  const int64_t ring_base = static_cast<int64_t>(b) * p.ring_vec_per_stream +
                            (static_cast<int64_t>(slot) * p.T + t) * p.vec_per_token;
  const int64_t tab_base = (static_cast<int64_t>(b) * p.table_stream_stride >> 2) +
                           static_cast<int64_t>(n) * (kPairs / 4);

  double sq = 0.0, sk = 0.0;
  {
    // four vectors of q and of k per lane in flight at a time
    for (int v0 = lane; v0 < p.vec_per_token; v0 += 32 * 4) {
      uint4 xq[4], xk[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int vi = v0 + 32 * u;
        if (vi < p.vec_per_token) {
          xq[u] = q_in[in_base + vi];   // plain load: q_out may be the same buffer
          xk[u] = __ldg(k_in + in_base + vi);
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (v0 + 32 * u < p.vec_per_token) {
          sq = squares(xq[u], sq);
          sk = squares(xk[u], sk);
        }
      }
    }
  }
  const double width = static_cast<double>(p.vec_per_token) * 8.0;
  const float ms_q = static_cast<float>(warp_sum(sq) / width), ms_k = static_cast<float>(warp_sum(sk) / width);
  const float rq = __frcp_rn(__fsqrt_rn(__fadd_rn(ms_q, eps)));
  const float rk = __frcp_rn(__fsqrt_rn(__fadd_rn(ms_k, eps)));

  auto finish = [&](int vi, uint4 xq, uint4 xk) {
    const float4 c = __ldg(cos_t + tab_base + (vi & 15));
    const float4 s = __ldg(sin_t + tab_base + (vi & 15));
    const uint4 nq = normalise_vec(xq, rq, __ldg(gain_q + 2 * vi), __ldg(gain_q + 2 * vi + 1));
    const uint4 nk = normalise_vec(xk, rk, __ldg(gain_k + 2 * vi), __ldg(gain_k + 2 * vi + 1));
    UNSTEP_STORE(q_out, in_base + vi, p.extent_act, rotate_vec(nq, c, s), p.status);
    UNSTEP_STORE(ring_k, ring_base + vi, p.extent_cache, rotate_vec(nk, c, s), p.status);
    UNSTEP_STORE(ring_v, ring_base + vi, p.extent_cache, __ldcs(v_in + in_base + vi), p.status);
  };
  {
    for (int v0 = lane; v0 < p.vec_per_token; v0 += 32 * 2) {
      uint4 xq[2], xk[2];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int vi = v0 + 32 * u;
        if (vi < p.vec_per_token) {
          xq[u] = q_in[in_base + vi];
          xk[u] = k_in[in_base + vi];
        }
      }
#pragma unroll
      for (int u = 0; u < 2; ++u)
        if (v0 + 32 * u < p.vec_per_token) finish(v0 + 32 * u, xq[u], xk[u]);
    }
  }
}


// One thread block per token, for token vectors of up to 4 * 256 vectors (64 heads): thread i
// owns vectors i, i + blockDim, ... (kU of them) of q, k and v, all of them loaded at once and
// kept in registers from the sum of squares to the rotated store, so that a token makes one
// trip to memory.  The partial sums meet in shared memory and every thread adds them in the
// same order.
template <int kU>
__global__ void __launch_bounds__(kU <= 2 ? 96 : 256, kU <= 2 ? 12 : 3)
rmsnorm_rope_kv_append_token_kernel(AppendParams p, float eps, const uint4* q_in, const uint4* __restrict__ k_in,
                                    const uint4* __restrict__ v_in, const float4* __restrict__ gain_q,
                                    const float4* __restrict__ gain_k, const float4* __restrict__ cos_t,
                                    const float4* __restrict__ sin_t, uint4* q_out, uint4* __restrict__ ring_k,
                                    uint4* __restrict__ ring_v) {
  __shared__ double part[2][8];
  const int b = blockIdx.y;
  const int n = blockIdx.x;   // token
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int f = n / p.T, t = n - f * p.T;
  const int frame = p.start[b] + f;
  const int slot = frame < p.S ? frame : p.S + (frame - p.S) % p.C;
  const int64_t in_base = static_cast<int64_t>(b) * p.vec_per_stream + static_cast<int64_t>(n) * p.vec_per_token;
  const int64_t ring_base = static_cast<int64_t>(b) * p.ring_vec_per_stream +
                            (static_cast<int64_t>(slot) * p.T + t) * p.vec_per_token;
  const int64_t tab_base = (static_cast<int64_t>(b) * p.table_stream_stride >> 2) +
                           static_cast<int64_t>(n) * (kPairs / 4);

  uint4 xq[kU], xk[kU], xv[kU];
#pragma unroll
  for (int u = 0; u < kU; ++u) {
    const int vi = tid + u * nthr;
    if (vi < p.vec_per_token) {
      xq[u] = q_in[in_base + vi];   // plain load: q_out may be the same buffer
      xk[u] = __ldcs(k_in + in_base + vi);
      xv[u] = __ldcs(v_in + in_base + vi);
    }
  }
  // All vectors of a thread sit at the same place of their heads (the block is a multiple of 16
  // threads wide), so they share one set of coefficients, fetched under the wait for q, k and v.
  const float4 c = __ldg(cos_t + tab_base + (tid & 15));
  const float4 s = __ldg(sin_t + tab_base + (tid & 15));
  double sq = 0.0, sk = 0.0;
#pragma unroll
  for (int u = 0; u < kU; ++u) {
    const int vi = tid + u * nthr;
    if (vi < p.vec_per_token) {
      sq = squares(xq[u], sq);
      sk = squares(xk[u], sk);
      UNSTEP_STORE(ring_v, ring_base + vi, p.extent_cache, xv[u], p.status);
    }
  }
  sq = warp_sum(sq);
  sk = warp_sum(sk);
  if ((tid & 31) == 0) {
    part[0][tid >> 5] = sq;
    part[1][tid >> 5] = sk;
  }
  __syncthreads();
  // even lanes finish q, odd lanes k: one division per warp
  double tot = 0.0;
  for (int w = 0; w < (nthr >> 5); ++w) tot += part[tid & 1][w];
  const double width = static_cast<double>(p.vec_per_token) * 8.0;
  const float ms = static_cast<float>(tot / width);
  const float r = __frcp_rn(__fsqrt_rn(__fadd_rn(ms, eps)));
  const float rq = __shfl_sync(0xFFFFFFFFu, r, 0), rk = __shfl_sync(0xFFFFFFFFu, r, 1);
#pragma unroll
  for (int u = 0; u < kU; ++u) {
    const int vi = tid + u * nthr;
    if (vi < p.vec_per_token) {
      const uint4 nq = normalise_vec(xq[u], rq, __ldg(gain_q + 2 * vi), __ldg(gain_q + 2 * vi + 1));
      const uint4 nk = normalise_vec(xk[u], rk, __ldg(gain_k + 2 * vi), __ldg(gain_k + 2 * vi + 1));
      UNSTEP_STORE(q_out, in_base + vi, p.extent_act, rotate_vec(nq, c, s), p.status);
      UNSTEP_STORE(ring_k, ring_base + vi, p.extent_cache, rotate_vec(nk, c, s), p.status);
    }
  }
}

}  // namespace unstep

using namespace unstep;

extern "C" int unstep_rope_table(const unstep_shape_t* shape, int32_t start_frame, float* cos_out,
                                 float* sin_out, void* cuda_stream) {
  int rc = check_shape(shape, false);
  if (rc != UNSTEP_OK) return rc;
  if (start_frame < 0 || cos_out == nullptr || sin_out == nullptr) return UNSTEP_ERR_INVALID_ARG;
  if (!aligned16(cos_out) || !aligned16(sin_out)) return UNSTEP_ERR_INVALID_ARG;
  rc = check_device();
  if (rc != UNSTEP_OK) return rc;
  TableParams p;
  p.start_frame = start_frame;
  p.grid_h = shape->grid_h;
  p.grid_w = shape->grid_w;
  p.L = shape->chunk_frames * shape->grid_h * shape->grid_w;
  p.pairs_t = shape->band_t / 2;
  p.pairs_h = shape->band_h / 2;
  p.band_t = shape->band_t;
  p.band_h = shape->band_h;
  p.band_w = shape->band_w;
  p.base = shape->rope_base;
  p.status = status_word();
  p.extent = static_cast<int64_t>(p.L) * kPairs;
  if (shape->chunk_frames > 65535) return UNSTEP_ERR_INVALID_ARG;
  rope_table_kernel<<<dim3(shape->grid_h, shape->chunk_frames), 1024, 0,
                      static_cast<cudaStream_t>(cuda_stream)>>>(p, cos_out, sin_out);
  g_launches.fetch_add(1);
  return cudaGetLastError() == cudaSuccess ? UNSTEP_OK : UNSTEP_ERR_CUDA;
}

static int rope_kv_append_run(const unstep_shape_t* shape, int32_t sink_frames,
                              const int32_t* start_frame, const void* q_in, const void* k_in,
                              const void* v_in, const float* cos, const float* sin,
                              int64_t table_stream_stride, void* q_out, void* ring_k, void* ring_v,
                              void* cuda_stream) {
  int rc = check_shape(shape, true);
  if (rc != UNSTEP_OK) return rc;
  if (sink_frames < 0 || sink_frames > 4096) return UNSTEP_ERR_INVALID_ARG;
  const void* ptrs[] = {start_frame, q_in, k_in, v_in, cos, sin, q_out, ring_k, ring_v};
  for (const void* ptr : ptrs)
    if (ptr == nullptr) return UNSTEP_ERR_INVALID_ARG;
  const void* dev_ptrs[] = {q_in, k_in, v_in, cos, sin, q_out, ring_k, ring_v};
  for (const void* ptr : dev_ptrs)
    if (!aligned16(ptr)) return UNSTEP_ERR_INVALID_ARG;
  if (table_stream_stride < 0 || (table_stream_stride & 3)) return UNSTEP_ERR_INVALID_ARG;
  for (int b = 0; b < shape->batch; ++b)
    if (start_frame[b] < 0 || start_frame[b] > INT32_MAX - shape->chunk_frames) return UNSTEP_ERR_INVALID_ARG;
  rc = check_device();
  if (rc != UNSTEP_OK) return rc;

  const int64_t T = static_cast<int64_t>(shape->grid_h) * shape->grid_w;
  const int64_t L = T * shape->chunk_frames;
  AppendParams p;
  p.L = static_cast<int32_t>(L);
  p.T = static_cast<int32_t>(T);
  p.C = shape->ring_frames;
  p.S = sink_frames;
  p.vec_per_token = shape->heads * 16;
  p.vec_per_stream = L * p.vec_per_token;
  p.ring_vec_per_stream = (static_cast<int64_t>(shape->ring_frames) + sink_frames) * T * p.vec_per_token;
  p.table_stream_stride = table_stream_stride;
  const unsigned blocks = static_cast<unsigned>((p.vec_per_stream + 255) / 256);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  for (int b0 = 0; b0 < shape->batch; b0 += kMaxStreamsPerLaunch) {
    const int nb = shape->batch - b0 < kMaxStreamsPerLaunch ? shape->batch - b0 : kMaxStreamsPerLaunch;
    for (int i = 0; i < nb; ++i) p.start[i] = start_frame[b0 + i];
    p.status = status_word();
    p.extent_act = nb * p.vec_per_stream;
    p.extent_cache = nb * p.ring_vec_per_stream;
    const int64_t in_off = static_cast<int64_t>(b0) * p.vec_per_stream;
    const int64_t ring_off = static_cast<int64_t>(b0) * p.ring_vec_per_stream;
    const int64_t tab_off = static_cast<int64_t>(b0) * table_stream_stride;
    rope_kv_append_kernel<<<dim3(blocks, nb), 256, 0, st>>>(
        p, static_cast<const uint4*>(q_in) + in_off, static_cast<const uint4*>(k_in) + in_off,
        static_cast<const uint4*>(v_in) + in_off, reinterpret_cast<const float4*>(cos + tab_off),
        reinterpret_cast<const float4*>(sin + tab_off), static_cast<uint4*>(q_out) + in_off,
        static_cast<uint4*>(ring_k) + ring_off, static_cast<uint4*>(ring_v) + ring_off);
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) return UNSTEP_ERR_CUDA;
  }
  return UNSTEP_OK;
}

extern "C" int unstep_rope_kv_append(const unstep_shape_t* shape, const int32_t* start_frame,
                                     const void* q_in, const void* k_in, const void* v_in,
                                     const float* cos, const float* sin,
                                     int64_t table_stream_stride, void* q_out, void* ring_k,
                                     void* ring_v, void* cuda_stream) {
  return rope_kv_append_run(shape, 0, start_frame, q_in, k_in, v_in, cos, sin, table_stream_stride,
                            q_out, ring_k, ring_v, cuda_stream);
}

extern "C" int unstep_rope_kv_append_sink(const unstep_shape_t* shape, int32_t sink_frames,
                                          const int32_t* start_frame, const void* q_in,
                                          const void* k_in, const void* v_in, const float* cos,
                                          const float* sin, int64_t table_stream_stride, void* q_out,
                                          void* cache_k, void* cache_v, void* cuda_stream) {
  return rope_kv_append_run(shape, sink_frames, start_frame, q_in, k_in, v_in, cos, sin,
                            table_stream_stride, q_out, cache_k, cache_v, cuda_stream);
}

extern "C" int unstep_rmsnorm_rope_kv_append(const unstep_shape_t* shape, int32_t sink_frames,
                                             const int32_t* start_frame, const void* q_in,
                                             const void* k_in, const void* v_in, const float* gain_q,
                                             const float* gain_k, float eps, const float* cos,
                                             const float* sin, int64_t table_stream_stride, void* q_out,
                                             void* cache_k, void* cache_v, void* cuda_stream) {
  int rc = check_shape(shape, true);
  if (rc != UNSTEP_OK) return rc;
  if (sink_frames < 0 || sink_frames > 4096 || !(eps >= 0.f)) return UNSTEP_ERR_INVALID_ARG;
  const void* ptrs[] = {start_frame, q_in, k_in, v_in, gain_q, gain_k, cos, sin, q_out, cache_k, cache_v};
  for (const void* ptr : ptrs)
    if (ptr == nullptr) return UNSTEP_ERR_INVALID_ARG;
  const void* dev_ptrs[] = {q_in, k_in, v_in, gain_q, gain_k, cos, sin, q_out, cache_k, cache_v};
  for (const void* ptr : dev_ptrs)
    if (!aligned16(ptr)) return UNSTEP_ERR_INVALID_ARG;
  if (table_stream_stride < 0 || (table_stream_stride & 3)) return UNSTEP_ERR_INVALID_ARG;
  for (int b = 0; b < shape->batch; ++b)
    if (start_frame[b] < 0 || start_frame[b] > INT32_MAX - shape->chunk_frames) return UNSTEP_ERR_INVALID_ARG;
  rc = check_device();
  if (rc != UNSTEP_OK) return rc;

  const int64_t T = static_cast<int64_t>(shape->grid_h) * shape->grid_w;
  const int64_t L = T * shape->chunk_frames;
  AppendParams p;
  p.L = static_cast<int32_t>(L);
  p.T = static_cast<int32_t>(T);
  p.C = shape->ring_frames;
  p.S = sink_frames;
  p.vec_per_token = shape->heads * 16;
  p.vec_per_stream = L * p.vec_per_token;
  p.ring_vec_per_stream = (static_cast<int64_t>(shape->ring_frames) + sink_frames) * T * p.vec_per_token;
  p.table_stream_stride = table_stream_stride;
  const unsigned blocks = static_cast<unsigned>((L + 7) / 8);   // 8 warps = 8 tokens per block
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  for (int b0 = 0; b0 < shape->batch; b0 += kMaxStreamsPerLaunch) {
    const int nb = shape->batch - b0 < kMaxStreamsPerLaunch ? shape->batch - b0 : kMaxStreamsPerLaunch;
    for (int i = 0; i < nb; ++i) p.start[i] = start_frame[b0 + i];
    p.status = status_word();
    p.extent_act = nb * p.vec_per_stream;
    p.extent_cache = nb * p.ring_vec_per_stream;
    const int64_t in_off = static_cast<int64_t>(b0) * p.vec_per_stream;
    const int64_t ring_off = static_cast<int64_t>(b0) * p.ring_vec_per_stream;
    const int64_t tab_off = static_cast<int64_t>(b0) * table_stream_stride;
    const uint4* q = static_cast<const uint4*>(q_in) + in_off;
    const uint4* k = static_cast<const uint4*>(k_in) + in_off;
    const uint4* v = static_cast<const uint4*>(v_in) + in_off;
    const float4* gq = reinterpret_cast<const float4*>(gain_q);
    const float4* gk = reinterpret_cast<const float4*>(gain_k);
    const float4* ct = reinterpret_cast<const float4*>(cos + tab_off);
    const float4* sn = reinterpret_cast<const float4*>(sin + tab_off);
    uint4* qo = static_cast<uint4*>(q_out) + in_off;
    uint4* rk = static_cast<uint4*>(cache_k) + ring_off;
    uint4* rv = static_cast<uint4*>(cache_v) + ring_off;
    // Up to 64 heads: a thread block per token, of few threads with several vectors each (about
    // 96 threads for the 12 heads of the 1.3B shape: more tokens in flight per SM than with wider
    // blocks, 21.6 against 26 us there).
    if (p.vec_per_token <= 4 * 256) {
      int per_thread = (p.vec_per_token + 95) / 96;
      if (per_thread > 4) per_thread = 4;
      const int threads = (((p.vec_per_token + per_thread - 1) / per_thread) + 31) & ~31;
      const dim3 grid(static_cast<unsigned>(L), nb);
      switch (per_thread) {
        case 1: rmsnorm_rope_kv_append_token_kernel<1><<<grid, threads, 0, st>>>(p, eps, q, k, v, gq, gk, ct, sn, qo, rk, rv); break;
        case 2: rmsnorm_rope_kv_append_token_kernel<2><<<grid, threads, 0, st>>>(p, eps, q, k, v, gq, gk, ct, sn, qo, rk, rv); break;
        case 3: rmsnorm_rope_kv_append_token_kernel<3><<<grid, threads, 0, st>>>(p, eps, q, k, v, gq, gk, ct, sn, qo, rk, rv); break;
        default: rmsnorm_rope_kv_append_token_kernel<4><<<grid, threads, 0, st>>>(p, eps, q, k, v, gq, gk, ct, sn, qo, rk, rv); break;
      }
      g_launches.fetch_add(1);
      if (cudaGetLastError() != cudaSuccess) return UNSTEP_ERR_CUDA;
      continue;
    }
    // wider tokens: one warp per token
    rmsnorm_rope_kv_append_kernel<<<dim3(blocks, nb), 256, 0, st>>>(p, eps, q, k, v, gq, gk, ct, sn, qo, rk, rv);
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) return UNSTEP_ERR_CUDA;
  }
  return UNSTEP_OK;
}
