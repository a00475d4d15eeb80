// Windowed attention of one chunk over the KV ring: TMA-staged tiles, tcgen05 MMA
// into TMEM for Q K^T and P V, online softmax in registers.
//
// Work item = (stream b, head h, 128-query tile).  Keys are walked frame by frame:
// frame p of the window lives in ring slot p mod C, and every 128-key tile lies
// inside one frame, so the 5-D tensor map (d, head, token, slot, stream) zero-fills
// the ragged end of a frame and the ring never has to be copied or linearised.
#include <cuda.h>
#include <cuda_bf16.h>

#include <mutex>

#include "common.h"
#include "ptx.cuh"

namespace unstep {

using namespace ptx;

__device__ int g_status = 0;

constexpr int kTileM = 128;          // queries per work item
constexpr int kTileN = 128;          // keys per tile
constexpr int kHalfBytes = 128 * 64 * 2;   // one TMA box: 128 rows x 64 bf16 (128-byte rows)
constexpr int kTileBytes = 2 * kHalfBytes; // 128 x 128 bf16
constexpr int kTmemCols = 256;       // S/P: columns [0,128), O: columns [128,256)
constexpr long long kWaitCycles = 2000000000LL;  // about a second: then give up, never hang

struct AttnParams {
  int32_t Hn, L, T, C;
  int32_t q_tiles;         // ceil(L / 128)
  int32_t tiles_per_frame; // ceil(T / 128)
  float scale_log2e;       // log2(e) / sqrt(128)
  int32_t first_frame[kMaxStreamsPerLaunch];  // first attended absolute frame of stream b
  int32_t n_frames[kMaxStreamsPerLaunch];     // attended frames of stream b
};

struct Waiter {
  volatile int* abort_flag;
  __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) const {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
      if (mbar_try_wait(bar, parity)) return true;
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) {
        *abort_flag = 1;
        atomicExch(&g_status, UNSTEP_ERR_TIMEOUT);
        return false;
      }
    }
  }
};

__global__ void __launch_bounds__(128, 2)
window_attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const AttnParams p,
                   __nv_bfloat16* __restrict__ out) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = smem_base;
  const uint32_t sK = sQ + kTileBytes;
  const uint32_t sV = sK + kTileBytes;
  const uint32_t sBar = sV + kTileBytes;
  const uint32_t bar_q = sBar + 0, bar_k = sBar + 8, bar_v = sBar + 16, bar_s = sBar + 24,
                 bar_o = sBar + 32;
  uint8_t* gen = smem_raw + (smem_base - smem_u32(smem_raw)) + 3 * kTileBytes;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + 64);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + 72);

  const int tid = threadIdx.x;
  const int warp = tid >> 5;

  // work item: q tile fastest, then head, then stream, so neighbouring CTAs share K/V in L2
  int item = blockIdx.x;
  const int qt = item % p.q_tiles;
  item /= p.q_tiles;
  const int h = item % p.Hn;
  const int b = item / p.Hn;
  const int n0 = qt * kTileM;
  const int first_frame = p.first_frame[b];
  const int total_tiles = p.n_frames[b] * p.tiles_per_frame;

  if (tid == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_k, 1);
    mbar_init(bar_v, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_o, 1);
    *abort_flag = 0;
    mbar_fence_init();
    prefetch_tensormap(&tm_q);
    prefetch_tensormap(&tm_k);
    prefetch_tensormap(&tm_v);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
  const uint32_t t_S = t_lane;        // this warp's 32 lanes, columns [0, 128)
  const uint32_t t_O = t_lane + 128;  // columns [128, 256)
  const Waiter w{abort_flag};

  constexpr uint32_t kIdescQK = idesc_bf16_f32(kTileM, kTileN, 0);
  constexpr uint32_t kIdescPV = idesc_bf16_f32(kTileM, kHeadDim, 1);

  auto issue_kv_load = [&](uint32_t dst, const CUtensorMap* tm, uint32_t bar, int j) {
    const int fi = j / p.tiles_per_frame;
    const int tok0 = (j - fi * p.tiles_per_frame) * kTileN;
    const int slot = (first_frame + fi) % p.C;
    mbar_expect_tx(bar, kTileBytes);
    tma_load_5d(dst, tm, bar, 0, h, tok0, slot, b);
    tma_load_5d(dst + kHalfBytes, tm, bar, 64, h, tok0, slot, b);
  };

  bool k_inflight = false, v_inflight = false, q_inflight = false;
  if (tid == 0) {
    mbar_expect_tx(bar_q, kTileBytes);
    tma_load_4d(sQ, &tm_q, bar_q, 0, h, n0, b);
    tma_load_4d(sQ + kHalfBytes, &tm_q, bar_q, 64, h, n0, b);
    issue_kv_load(sK, &tm_k, bar_k, 0);
    issue_kv_load(sV, &tm_v, bar_v, 0);
    q_inflight = k_inflight = v_inflight = true;
  }

  float m_run = -INFINITY, l_run = 0.f;
  bool ok = true;

  for (int j = 0; j < total_tiles && ok; ++j) {
    const uint32_t ph = j & 1;
    const int fi = j / p.tiles_per_frame;
    const int tok0 = (j - fi * p.tiles_per_frame) * kTileN;
    const int nvalid = min(kTileN, p.T - tok0);

    // ---- S = Q K^T -------------------------------------------------------
    if (tid == 0) {
      if (j == 0) {
        ok = w.wait(bar_q, 0);
        q_inflight = false;
      }
      if (ok) ok = w.wait(bar_k, ph);
      if (ok) {
        k_inflight = false;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t off = (k >> 2) * kHalfBytes + (k & 3) * 32;
          mma_ss(tmem_base, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024),
                 kIdescQK, k > 0);
        }
        tc_commit(bar_s);
      }
    }
    if (!w.wait(bar_s, ph)) { ok = false; break; }
    tc_fence_after();
    if (tid == 0 && j + 1 < total_tiles) {  // K tile is consumed: prefetch the next one
      issue_kv_load(sK, &tm_k, bar_k, j + 1);
      k_inflight = true;
    }

    // ---- online softmax on this thread's row ----------------------------
    uint32_t sreg[128];
#pragma unroll
    for (int c = 0; c < 4; ++c) tmem_ld32(t_S + c * 32, sreg + c * 32);
    tc_wait_ld();
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < 128; ++i) {
      float s = __uint_as_float(sreg[i]);
      if (i >= nvalid) s = -INFINITY;
      sreg[i] = __float_as_uint(s);
      mx = fmaxf(mx, s);
    }
    const float m_new = fmaxf(m_run, mx);
    const float alpha = ex2((m_run - m_new) * p.scale_log2e);
    const float neg_ms = -m_new * p.scale_log2e;
    float psum = 0.f;
    // P (bf16, two per column) overwrites the first 64 columns of S, 32 columns at a time
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t preg[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float p0 = ex2(fmaf(__uint_as_float(sreg[64 * half + 2 * i]), p.scale_log2e, neg_ms));
        const float p1 = ex2(fmaf(__uint_as_float(sreg[64 * half + 2 * i + 1]), p.scale_log2e, neg_ms));
        psum += p0 + p1;
        preg[i] = pack_bf16x2(p0, p1);
      }
      tmem_st32(t_S + 32 * half, preg);
    }
    l_run = fmaf(l_run, alpha, psum);
    m_run = m_new;
    // rescale the running output when some row of the warp moved its maximum
    if (j > 0 && __any_sync(0xFFFFFFFFu, alpha != 1.f)) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t o[32];
        tmem_ld32(t_O + c * 32, o);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
        tmem_st32(t_O + c * 32, o);
      }
    }
    tc_wait_st();
    tc_fence_before();
    __syncthreads();

    // ---- O += P V ---------------------------------------------------------
    if (tid == 0) {
      tc_fence_after();
      ok = w.wait(bar_v, ph);
      if (ok) {
        v_inflight = false;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          mma_ts(tmem_base + 128, tmem_base + k * 8, smem_desc_sw128(sV + k * 2048, kHalfBytes, 1024),
                 kIdescPV, (j > 0 || k > 0) ? 1u : 0u);
        }
        tc_commit(bar_o);
      }
    }
    if (!w.wait(bar_o, ph)) { ok = false; break; }
    tc_fence_after();
    if (tid == 0 && j + 1 < total_tiles) {  // V tile is consumed: prefetch the next one
      issue_kv_load(sV, &tm_v, bar_v, j + 1);
      v_inflight = true;
    }
  }

  // ---- epilogue: O / l -> bf16 -> out[b][n][h][:] -------------------------
  if (!*abort_flag) {
    const int n = n0 + tid;
    const float inv_l = 1.f / l_run;
    uint4* dst = reinterpret_cast<uint4*>(out + ((static_cast<int64_t>(b) * p.L + n) * p.Hn + h) * kHeadDim);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      uint32_t o[32];
      tmem_ld32(t_O + c * 32, o);
      tc_wait_ld();
      if (n < p.L) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint4 vv;
          vv.x = pack_bf16x2(__uint_as_float(o[8 * i + 0]) * inv_l, __uint_as_float(o[8 * i + 1]) * inv_l);
          vv.y = pack_bf16x2(__uint_as_float(o[8 * i + 2]) * inv_l, __uint_as_float(o[8 * i + 3]) * inv_l);
          vv.z = pack_bf16x2(__uint_as_float(o[8 * i + 4]) * inv_l, __uint_as_float(o[8 * i + 5]) * inv_l);
          vv.w = pack_bf16x2(__uint_as_float(o[8 * i + 6]) * inv_l, __uint_as_float(o[8 * i + 7]) * inv_l);
          dst[c * 4 + i] = vv;
        }
      }
    }
  } else if (tid == 0) {
    // gave up: let this CTA's own copies land (bounded) before the shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {
      const bool q_done = !q_inflight || mbar_try_wait(bar_q, 0);
      const bool k_done = !k_inflight || mbar_try_wait(bar_k, 0) || mbar_try_wait(bar_k, 1);
      const bool v_done = !v_inflight || mbar_try_wait(bar_v, 0) || mbar_try_wait(bar_v, 1);
      if (q_done && k_done && v_done) break;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, kTmemCols);
}

// --------------------------------------------------------------------------
// Host side
// --------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  });
  return fn;
}

// bf16 tensor map with 128-byte swizzle, box = 64 elements x 128 rows of dimension `row_dim`.
static bool make_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims,
                     const uint64_t* strides_bytes, int row_dim) {
  EncodeTiledFn fn = get_encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t gdim[5], gstride[4];
  cuuint32_t box[5], estr[5];
  for (int i = 0; i < rank; ++i) {
    gdim[i] = dims[i];
    box[i] = 1;
    estr[i] = 1;
    if (i > 0) gstride[i - 1] = strides_bytes[i - 1];
  }
  box[0] = 64;
  box[row_dim] = 128;
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kAttnSmemBytes = 3 * kTileBytes + 1024 + 128;

}  // namespace unstep

using namespace unstep;

extern "C" int unstep_window_attn(const unstep_shape_t* shape, const int32_t* start_frame,
                                  int32_t window_frames, const void* q_rot, const void* ring_k,
                                  const void* ring_v, void* out, void* cuda_stream) {
  int rc = check_shape(shape, true);
  if (rc != UNSTEP_OK) return rc;
  const void* ptrs[] = {start_frame, q_rot, ring_k, ring_v, out};
  for (const void* ptr : ptrs)
    if (ptr == nullptr) return UNSTEP_ERR_INVALID_ARG;
  if (!aligned16(q_rot) || !aligned16(ring_k) || !aligned16(ring_v) || !aligned16(out))
    return UNSTEP_ERR_INVALID_ARG;
  if (window_frames < shape->chunk_frames || window_frames > shape->ring_frames)
    return UNSTEP_ERR_INVALID_ARG;
  for (int b = 0; b < shape->batch; ++b)
    if (start_frame[b] < 0 || start_frame[b] > INT32_MAX - shape->chunk_frames)
      return UNSTEP_ERR_INVALID_ARG;
  rc = check_device();
  if (rc != UNSTEP_OK) return rc;

  static std::once_flag attr_once;
  static bool attr_ok = false;
  std::call_once(attr_once, [] {
    attr_ok = cudaFuncSetAttribute(window_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   kAttnSmemBytes) == cudaSuccess;
  });
  if (!attr_ok) return UNSTEP_ERR_CUDA;

  const uint64_t Hn = shape->heads, C = shape->ring_frames;
  const uint64_t T = static_cast<uint64_t>(shape->grid_h) * shape->grid_w;
  const uint64_t L = T * shape->chunk_frames;
  const uint64_t row_bytes = Hn * kHeadDim * 2;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

  AttnParams p;
  p.Hn = shape->heads;
  p.L = static_cast<int32_t>(L);
  p.T = static_cast<int32_t>(T);
  p.C = shape->ring_frames;
  p.q_tiles = static_cast<int32_t>((L + kTileM - 1) / kTileM);
  p.tiles_per_frame = static_cast<int32_t>((T + kTileN - 1) / kTileN);
  p.scale_log2e = 1.4426950408889634f / sqrtf(static_cast<float>(kHeadDim));

  for (int b0 = 0; b0 < shape->batch; b0 += kMaxStreamsPerLaunch) {
    const int nb = shape->batch - b0 < kMaxStreamsPerLaunch ? shape->batch - b0 : kMaxStreamsPerLaunch;
    for (int i = 0; i < nb; ++i) {
      const int hi = start_frame[b0 + i] + shape->chunk_frames;
      const int lo = hi - window_frames > 0 ? hi - window_frames : 0;
      p.first_frame[i] = lo;
      p.n_frames[i] = hi - lo;
    }
    const char* qb = static_cast<const char*>(q_rot) + static_cast<uint64_t>(b0) * L * row_bytes;
    const char* kb = static_cast<const char*>(ring_k) + static_cast<uint64_t>(b0) * C * T * row_bytes;
    const char* vb = static_cast<const char*>(ring_v) + static_cast<uint64_t>(b0) * C * T * row_bytes;
    __nv_bfloat16* ob = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(out) +
                                                         static_cast<uint64_t>(b0) * L * row_bytes);
    CUtensorMap tm_q, tm_k, tm_v;
    const uint64_t qdims[4] = {kHeadDim, Hn, L, static_cast<uint64_t>(nb)};
    const uint64_t qstr[3] = {kHeadDim * 2, row_bytes, L * row_bytes};
    const uint64_t rdims[5] = {kHeadDim, Hn, T, C, static_cast<uint64_t>(nb)};
    const uint64_t rstr[4] = {kHeadDim * 2, row_bytes, T * row_bytes, C * T * row_bytes};
    if (!make_map(&tm_q, qb, 4, qdims, qstr, 2) || !make_map(&tm_k, kb, 5, rdims, rstr, 2) ||
        !make_map(&tm_v, vb, 5, rdims, rstr, 2))
      return UNSTEP_ERR_CUDA;
    const unsigned grid = static_cast<unsigned>(nb) * p.Hn * p.q_tiles;
    window_attn_kernel<<<grid, 128, kAttnSmemBytes, st>>>(tm_q, tm_k, tm_v, p, ob);
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) return UNSTEP_ERR_CUDA;
  }
  return UNSTEP_OK;
}

extern "C" int unstep_poll_status(void) {
  if (cudaDeviceSynchronize() != cudaSuccess) return UNSTEP_ERR_CUDA;
  int st = 0, zero = 0;
  if (cudaMemcpyFromSymbol(&st, g_status, sizeof(int)) != cudaSuccess) return UNSTEP_ERR_CUDA;
  if (st != 0 && cudaMemcpyToSymbol(g_status, &zero, sizeof(int)) != cudaSuccess) return UNSTEP_ERR_CUDA;
  return st;
}
