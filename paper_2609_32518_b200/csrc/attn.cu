// Windowed attention of one chunk over the KV ring (sm_100a).
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warps 0-3   softmax of query tile 0, one thread per query row
//   warps 4-7   softmax of query tile 1
//   warp  8, 9  tcgen05.mma issuers of query tile 0 and 1 (one lane each); warp 8 owns TMEM
//   warp  10    TMA producer (one lane)
// A work item is (stream, head, pair of 128-query tiles): both tiles share every K/V
// tile.  The two tiles run half a period apart: while one is in its exponentials (MUFU
// pipe) the other's P V and next Q K^T run on the tensor core.  A small token ring keeps
// them apart: the MMA issuers take turns on the tensor pipe.  S = Q K^T and O += P V
// accumulate in TMEM; P (bf16) is written back over S and fed to the second MMA straight
// from TMEM.
//
// The attended frames are at most three runs of consecutive cache slots (sink prefix, ring
// up to its end, ring from its start).  Key tiles are cut from the runs through a flat
// tensor map over cache rows; only the last tile of a run is ragged, and it is fetched
// through a (token, slot) map whose zero fill ends it exactly at the end of its frame, so
// the cache is never copied and slots outside the window may hold anything.  A ragged tile
// runs with a narrower MMA (N and K rounded up to 16).
#include <cuda.h>
#include <cuda_bf16.h>

#include <map>
#include <mutex>
#include <utility>

#include "common.h"
#include "ptx.cuh"
#include "attn_sched.h"

namespace unstep {

using namespace ptx;

__device__ int g_status = 0;

// Optional timeline of CTA 0 (debug builds only): clock64 stamps per role, tile and event.
#ifdef UNSTEP_TRACE
__device__ long long g_trace[12][64][8];
__device__ unsigned long long g_cta_trace[160][16];
__device__ __forceinline__ unsigned long long gtime() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
#define CTRACE(ev)                                                                       \
  do {                                                                                   \
    if (threadIdx.x == 0 && (ev) < 16) g_cta_trace[blockIdx.x][ev] = gtime();            \
  } while (0)
#define TRACE(role, tile, ev)                                                          \
  do {                                                                                 \
    if (blockIdx.x == 0 && (tile) < 64 && (threadIdx.x & 31) == 0) {                   \
      const int w_ = threadIdx.x >> 5;                                                 \
      const int slot_ = (role) < 2 ? (w_ & 3) * 2 + (role) : 8 + (role) - 2;            \
      g_trace[slot_][tile][ev] = clock64();                                            \
    }                                                                                  \
  } while (0)
#else
#define TRACE(role, tile, ev) \
  do {                        \
  } while (0)
#define CTRACE(ev) \
  do {             \
  } while (0)
#endif

constexpr int kHalfBytes = 128 * 64 * 2;    // one TMA box: 128 rows x 64 bf16 (128-byte rows)
constexpr int kTileBytes = 2 * kHalfBytes;  // 128 x 128 bf16
constexpr int kStages = 5;                  // 32 KB buffers shared by the K and V tiles
constexpr int kThreads = 384;
constexpr int kTmemCols = 512;              // S0 | S1 | O0 | O1, 128 fp32 columns each
constexpr long long kWaitCycles = 2000000000LL;  // about a second: then give up, never hang

constexpr int kSmemQ = 0;
constexpr int kSmemKV = 2 * kTileBytes;
constexpr int kSmemBar = kSmemKV + kStages * kTileBytes;
constexpr int kAttnSmemBytes = kSmemBar + 256;

// Partial result of one query tile of a split item: O[col][row] (unnormalised, relative to the
// part's own reference maximum), then m[row], l[row].  Two tiles per slot, two slots per CTA.
constexpr int kPartTileFloats = 128 * 128 + 2 * 128;
constexpr int kPartFloats = 2 * kPartTileFloats;
struct Waiter {
  volatile int* abort_flag;
  long long limit;   // clock cycles after which a wait gives up
  // Bounded wait: the hardware parks the thread between polls; the clock and the CTA's abort
  // flag are only looked at every 32 polls so that a waiting warp leaves the issue slots alone.
  __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) const {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t spin = 1;; ++spin) {
      if (mbar_try_wait_hint(bar, parity, 2000u)) return true;
      if ((spin & 31u) == 0u) {
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
          *abort_flag = 1;
          atomicExch(&g_status, UNSTEP_ERR_TIMEOUT);
          return false;
        }
      }
    }
  }
};

// The CTA owns 384 x 168 registers; 128 x 72 for the service warps + 256 x 216 for the softmax
// warps uses exactly that (an increase that the pool cannot satisfy would wait forever).  216 is
// what the softmax warps need to run without spills.
constexpr int kRegsService = 72, kRegsSoftmax = 216;
static_assert(128 * kRegsService + 256 * kRegsSoftmax <= 384 * 168, "register redistribution exceeds the CTA's allocation");
static_assert(kRegsService == 72 && kRegsSoftmax == 216, "keep the setmaxnreg literals below in step");
__device__ __forceinline__ void reg_dealloc_service() { asm volatile("setmaxnreg.dec.sync.aligned.u32 72;"); }
__device__ __forceinline__ void reg_alloc_softmax() { asm volatile("setmaxnreg.inc.sync.aligned.u32 216;"); }

// --------------------------------------------------------------------------------------
// Softmax of one 128 x 128 score tile with one thread per query row (a warpgroup per query
// tile); no data crosses threads.  The caller has seen S of this tile complete, which (the
// tensor pipe runs in issue order) also means the previous P V into O has landed, so O may be
// rescaled here without another wait.
// --------------------------------------------------------------------------------------
__device__ __forceinline__ void group_barrier(int a) {
  if (a == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
  else asm volatile("bar.sync 2, 128;" ::: "memory");
}

// Exponentials of 32 score columns (registers s) into 16 bf16 pairs (p) and the packed sums.
__device__ __forceinline__ void exp_block32(const uint32_t* s, uint32_t* p, uint64_t c2, uint64_t nm2,
                                            uint64_t* acc) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const uint64_t x2 = fma_f32x2(pack_f32x2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), c2, nm2);
    float x0, x1;
    unpack_f32x2(x2, x0, x1);
    const float p0 = ex2(x0), p1 = ex2(x1);
    acc[i & 3] = add_f32x2(acc[i & 3], pack_f32x2(p0, p1));
    p[i] = pack_bf16x2(p0, p1);
  }
}
__device__ __forceinline__ float max_block32(const uint32_t* s) {
  float m = fmaxf(__uint_as_float(s[0]), __uint_as_float(s[1]));
#pragma unroll
  for (int i = 2; i < 32; i += 2) m = max3(m, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
  return m;
}
template <bool kMasked>
__device__ __forceinline__ void mask_block32(uint32_t* s, int col0, int nvalid) {
  if (kMasked) {
#pragma unroll
    for (int i = 0; i < 32; ++i)
      if (col0 + i >= nvalid) s[i] = 0xFF800000u;  // -inf
  }
}

// Exponentials of the 128 scores of a row (TMEM columns t_S .. t_S + 127) against the reference
// maximum: the scores come in blocks of 32 columns, each fetched while the block before it is
// exponentiated (a block keeps the MUFU pipe busy for 256 clk, longer than a TMEM load takes), so
// that only the first block's load is exposed.  Leaves P (bf16 pairs) in p0 (keys 0..63) and p1
// (keys 64..127) and returns the row's sum of P.
template <bool kMasked>
__device__ __forceinline__ float exp_row(uint32_t t_S, float c, float neg_ms, int nvalid, uint32_t* p0,
                                         uint32_t* p1) {
  const uint64_t c2 = pack_f32x2(c, c);
  const uint64_t nm2 = pack_f32x2(neg_ms, neg_ms);
  uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
  uint32_t a[32], b[32];
  tmem_ld32(t_S, a);
  tc_wait_ld32(a);
  tmem_ld32(t_S + 32, b);
  mask_block32<kMasked>(a, 0, nvalid);
  exp_block32(a, p0, c2, nm2, acc);
  tc_wait_ld32(b);
  tmem_ld32(t_S + 64, a);
  mask_block32<kMasked>(b, 32, nvalid);
  exp_block32(b, p0 + 16, c2, nm2, acc);
  tc_wait_ld32(a);
  tmem_ld32(t_S + 96, b);
  mask_block32<kMasked>(a, 64, nvalid);
  exp_block32(a, p1, c2, nm2, acc);
  tc_wait_ld32(b);
  mask_block32<kMasked>(b, 96, nvalid);
  exp_block32(b, p1 + 16, c2, nm2, acc);
  const uint64_t t = add_f32x2(add_f32x2(acc[0], acc[1]), add_f32x2(acc[2], acc[3]));
  float t0, t1;
  unpack_f32x2(t, t0, t1);
  return t0 + t1;
}

// Row maximum of the 128 scores in TMEM.
template <bool kMasked>
__device__ __forceinline__ float max_row(uint32_t t_S, int nvalid) {
  uint32_t hi[64], lo[64];
  tmem_ld32(t_S + 64, hi);
  tmem_ld32(t_S + 96, hi + 32);
  tmem_ld32(t_S, lo);
  tmem_ld32(t_S + 32, lo + 32);
  tc_wait_ld32(hi);
  reg_fence32(hi + 32);
  reg_fence32(lo);
  reg_fence32(lo + 32);
  mask_block32<kMasked>(hi, 64, nvalid);
  mask_block32<kMasked>(hi + 32, 96, nvalid);
  mask_block32<kMasked>(lo, 0, nvalid);
  mask_block32<kMasked>(lo + 32, 32, nvalid);
  return fmaxf(fmaxf(max_block32(hi), max_block32(hi + 32)), fmaxf(max_block32(lo), max_block32(lo + 32)));
}

// Only the first key tile of a segment looks for the row maximum before its exponentials.
// Every later tile exponentiates against that reference straight away and looks at the row's sum
// of P afterwards.  P is positive, so a sum of at most kOptimisticLimit = 2^64 means that no
// score was more than 64 (log2 units) above the reference: P (bf16) and the float32 sums are as
// accurate at that magnitude as near 1 (same relative precision, no overflow: 128 keys of 2^64
// times |v| stay far below 2^127), and everything accumulated before such a jump is negligible
// exactly as in the true softmax.  Otherwise (scores more than 64 above the first tile's maximum,
// or an overflow to inf) the warp finds the tile's true maximum, rescales O and l, and redoes
// the exponentials; the scores are still in TMEM, because P is only stored at the very end.
// Scores are read from TMEM in blocks to keep the register count down; P (bf16 pairs)
// overwrites score columns 0..63.
constexpr float kOptimisticLimit = 18446744073709551616.f;   // 2^64

template <bool kMasked>
__device__ __forceinline__ void softmax_row_tile(uint32_t t_S, uint32_t t_O, float c, int nvalid,
                                                 bool first, float& m_run, float& l_run,
                                                 uint32_t bar_p_full, int trace_role, int trace_tile) {
  if (first) m_run = max_row<kMasked>(t_S, nvalid);
  TRACE(trace_role, trace_tile, 2);
  uint32_t p0[32], p1[32];
  float sum = exp_row<kMasked>(t_S, c, -m_run * c, nvalid, p0, p1);
  const bool redo = !first && !(sum <= kOptimisticLimit);   // also taken for inf and NaN
  if (__any_sync(0xFFFFFFFFu, redo)) {
    const float mx = max_row<kMasked>(t_S, nvalid);
    float alpha = 1.f;
    if (mx > m_run) {
      alpha = ex2((m_run - mx) * c);
      m_run = mx;
      l_run *= alpha;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint32_t o[32];
      tmem_ld32(t_O + q * 32, o);
      tc_wait_ld32(o);
#pragma unroll
      for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
      tmem_st32(t_O + q * 32, o);
    }
    sum = exp_row<kMasked>(t_S, c, -m_run * c, nvalid, p0, p1);
  }
  tmem_st32(t_S, p0);        // P of keys 0..63 over score columns 0..31
  tmem_st32(t_S + 32, p1);   // P of keys 64..127 over score columns 32..63
  tc_wait_st();
  tc_fence_before();
  mbar_arrive(bar_p_full);
  TRACE(trace_role, trace_tile, 5);
  l_run += sum;
}

// Real keys of key tile j of a stream, without the divisions of tile_info: only the last tile of a
// run of slots is ragged (frames shorter than a tile: every tile is one frame).
struct ValidKeys {
  int j_last[3], v_last[3], dflt;
  __device__ __forceinline__ ValidKeys(const AttnParams& p, int b) {
    dflt = p.flat ? kTileN : p.T;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      const int begin = r == 0 ? 0 : p.run_tile_end[b][r - 1];
      const int end = p.run_tile_end[b][r];
      const bool any = p.flat && end > begin;
      j_last[r] = any ? end - 1 : -1;
      v_last[r] = p.run_rows[b][r] - kTileN * (end - begin - 1);
    }
  }
  __device__ __forceinline__ int operator()(int j) const {
    return j == j_last[0] ? v_last[0] : (j == j_last[1] ? v_last[1] : (j == j_last[2] ? v_last[2] : dflt));
  }
};

__global__ void __launch_bounds__(kThreads, 1)
window_attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kf,
                   const __grid_constant__ CUtensorMap tm_vf, const AttnParams p,
                   __nv_bfloat16* __restrict__ out) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = smem_u32(smem_raw);
  if (smem_base & 1023u) {  // the 128-byte swizzle needs 1024-byte aligned tiles
    if (threadIdx.x == 0) atomicExch(&g_status, UNSTEP_ERR_CUDA);
    return;
  }
  uint8_t* gen = smem_raw;
  const uint32_t sQ = smem_base + kSmemQ;
  const uint32_t sKV = smem_base + kSmemKV;
  const uint32_t sBar = smem_base + kSmemBar;
  // mbarriers (8 bytes each)
  const uint32_t bar_q_full = sBar;                          // [2]  TMA -> MMA warp a
  const uint32_t bar_q_empty = sBar + 16;                    // [2]  MMA warp a -> TMA
  const uint32_t bar_kv_full = sBar + 32;                    // [kStages] TMA -> both MMA warps
  const uint32_t bar_kv_empty = sBar + 32 + 8 * kStages;     // [kStages] both MMA warps -> TMA
  const uint32_t bar_s_full = sBar + 32 + 16 * kStages;      // [2]  MMA warp a -> softmax a
  const uint32_t bar_p_full = bar_s_full + 16;               // [2]  softmax a -> MMA warp a (128 arrivals)
  const uint32_t bar_o_final = bar_p_full + 16;              // [2]  MMA warp a -> softmax a
  const uint32_t bar_mturn = bar_o_final + 16;               // [2]  MMA warp 1-a -> MMA warp a: your turn on the tensor pipe
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + kSmemBar + 224);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + kSmemBar + 228);
  volatile int* merge_flag = reinterpret_cast<volatile int*>(gen + kSmemBar + 232);   // [2]

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  CTRACE(0);

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_q_full + 8 * i, 1);
      mbar_init(bar_q_empty + 8 * i, 1);
      mbar_init(bar_s_full + 8 * i, 1);
      mbar_init(bar_p_full + 8 * i, 128);
      mbar_init(bar_o_final + 8 * i, 1);
      mbar_init(bar_mturn + 8 * i, 1);
    }
    for (int i = 0; i < kStages; ++i) {
      mbar_init(bar_kv_full + 8 * i, 1);
      mbar_init(bar_kv_empty + 8 * i, 2);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 8) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const Waiter w{abort_flag, kWaitCycles};

  if (warp >= 8) {
    reg_dealloc_service();
    if (warp == 10 && lane == 0) {
      // ------------------------------------------------------------ TMA producer
      prefetch_tensormap(&tm_q);
      prefetch_tensormap(&tm_k);
      prefetch_tensormap(&tm_v);
      prefetch_tensormap(&tm_kf);
      prefetch_tensormap(&tm_vf);
      Sched sched(p, static_cast<int>(blockIdx.x));
      Seg s;
      uint32_t kv_it = 0, q_it[2] = {0, 0};
      bool ok = true;
      while (ok && sched.next(s)) {
        for (int a = 0; a < s.nq && ok; ++a) {
          ok = w.wait(bar_q_empty + 8 * a, (q_it[a] & 1) ^ 1);
          if (!ok) break;
          const uint32_t dst = sQ + a * kTileBytes, bar = bar_q_full + 8 * a;
          const int n0 = (2 * s.qp + a) * kTileM;
          mbar_expect_tx(bar, kTileBytes);
          tma_load_4d(dst, &tm_q, bar, 0, s.h, n0, s.b);
          tma_load_4d(dst + kHalfBytes, &tm_q, bar, 64, s.h, n0, s.b);
          ++q_it[a];
        }
        for (int j = s.t0; j < s.t1 && ok; ++j) {
          const TileInfo ti = tile_info(p, s.b, j);
          for (int kv = 0; kv < 2 && ok; ++kv) {
            const uint32_t st = kv_it % kStages;
            ok = w.wait(bar_kv_empty + 8 * st, ((kv_it / kStages) & 1) ^ 1);
            if (!ok) break;
            const uint32_t dst = sKV + st * kTileBytes, bar = bar_kv_full + 8 * st;
            mbar_expect_tx(bar, kTileBytes);
            if (ti.framed) {
              const CUtensorMap* tm = kv == 0 ? &tm_k : &tm_v;
              tma_load_5d(dst, tm, bar, 0, s.h, ti.tok0, ti.slot, s.b);
              tma_load_5d(dst + kHalfBytes, tm, bar, 64, s.h, ti.tok0, ti.slot, s.b);
            } else {
              const CUtensorMap* tm = kv == 0 ? &tm_kf : &tm_vf;
              tma_load_4d(dst, tm, bar, 0, s.h, ti.row, s.b);
              tma_load_4d(dst + kHalfBytes, tm, bar, 64, s.h, ti.row, s.b);
            }
            ++kv_it;
          }
        }
      }
    } else if (warp <= 9 && lane == 0) {
      // ------------------------------------------------------------ MMA issuer of query tile a
      // One issuing thread per query tile, on different scheduler partitions.  For each key
      // tile: O_a += P_a V (two halves, as P arrives), then S_a = Q_a K_next^T.  Both warps
      // walk the same K/V ring; a stage is released when both have retired it.
      const int a = warp - 8;
      Sched sched(p, static_cast<int>(blockIdx.x));
      Seg s;
      uint32_t kv_it = 0, q_it = 0, sp_it = 0, mturn_it = 0;
      bool ok = true;
      const uint32_t idesc_pv = idesc_bf16_f32(kTileM, kHeadDim, 1);
      const uint32_t idesc_qk_full = idesc_bf16_f32(kTileM, kTileN, 0);
      // descriptors are built once; per instruction only the start-address field moves
      const uint64_t dq = smem_desc_sw128(sQ + a * kTileBytes, 16, 1024);   // Q tile a, K-major
      const uint64_t dk0 = smem_desc_sw128(sKV, 16, 1024);                  // stage 0 as a K tile
      const uint64_t dv0 = smem_desc_sw128(sKV, kHalfBytes, 1024);          // stage 0 as a V tile (MN-major)
      const uint32_t s_tmem = tmem_base + a * 128, o_tmem = tmem_base + 256 + a * 128;
      const uint32_t my_s_full = bar_s_full + 8 * a, my_p_full = bar_p_full + 8 * a;

      // a ragged tile runs with N (for Q K^T) and K (for P V) rounded up to 16 keys
      auto issue_qk = [&](uint32_t stage, int valid) {
        const uint64_t dk = dk0 + static_cast<uint64_t>((stage * kTileBytes) >> 4);
        const uint32_t idesc = valid == kTileN ? idesc_qk_full : idesc_bf16_f32(kTileM, (valid + 15) & ~15, 0);
        mma_ss_k128(s_tmem, dq, dk, idesc, 0u);
        tc_commit(my_s_full);
        tc_commit(bar_kv_empty + 8 * stage);
      };
      auto issue_pv_half = [&](uint64_t dv, int half, int k_steps, bool accumulate) {
        if (k_steps >= 4 * half + 4) {
          mma_ts_k64(o_tmem, s_tmem + 32 * half, dv + static_cast<uint64_t>(512 * half), idesc_pv,
                     accumulate ? 1u : 0u);
          return;
        }
#pragma unroll
        for (int k = 4 * half; k < 4 * half + 4; ++k)
          if (k < k_steps)
            mma_ts(o_tmem, s_tmem + k * 8, dv + static_cast<uint64_t>((k * 2048) >> 4), idesc_pv,
                   (accumulate || k > 0) ? 1u : 0u);
      };

      while (ok && sched.next(s)) {
        const bool part = a < s.nq;   // a lone last query tile leaves warp 1 only the bookkeeping
        const int n = s.t1 - s.t0;
        const ValidKeys valid_of(p, s.b);
        int valid = valid_of(s.t0);  // real keys of the tile S is being computed for
        if (part) {
          ok = w.wait(bar_q_full + 8 * a, q_it & 1);
          if (!ok) break;
          ++q_it;
        }
        uint32_t kst = kv_it % kStages;
        ok = w.wait(bar_kv_full + 8 * kst, (kv_it / kStages) & 1);
        if (!ok) break;
        ++kv_it;
        if (part) {
          tc_fence_after();
          issue_qk(kst, valid);
          // Q is free as soon as the item's last Q K^T has run: the producer fetches the next
          // item's Q under this item's last exponentials and P V
          if (n == 1) tc_commit(bar_q_empty + 8 * a);
        } else {
          mbar_arrive(bar_kv_empty + 8 * kst);
        }
        for (int j = 0; j < n; ++j) {
          const int k_steps = (valid + 15) >> 4;
          const uint32_t vst = kv_it % kStages;
          ok = w.wait(bar_kv_full + 8 * vst, (kv_it / kStages) & 1);
          if (!ok) break;
          ++kv_it;
          const bool more = j + 1 < n;
          if (more) {
            valid = valid_of(s.t0 + j + 1);
            kst = kv_it % kStages;
            ok = w.wait(bar_kv_full + 8 * kst, (kv_it / kStages) & 1);
            if (!ok) break;
            ++kv_it;
          }
          if (part) {
            const uint64_t dv = dv0 + static_cast<uint64_t>((vst * kTileBytes) >> 4);
            TRACE(2 + a, sp_it, 0);
            ok = w.wait(my_p_full, sp_it & 1);   // P of this tile is in TMEM, O rescaled if need be
            if (!ok) break;
            TRACE(2 + a, sp_it, 1);
            // The two issuers take turns with their P V + Q K^T chains: issued side by side the
            // chains would interleave in the tensor pipe and finish together, which pulls the
            // two query tiles into step; one after the other keeps them half a period apart.
            if (s.nq == 2) {
              ok = w.wait(bar_mturn + 8 * a, (a == 0) ? ((mturn_it & 1) ^ 1) : (mturn_it & 1));
              if (!ok) break;
            }
            TRACE(2 + a, sp_it, 3);
            tc_fence_after();
            issue_pv_half(dv, 0, k_steps, j > 0);
            issue_pv_half(dv, 1, k_steps, true);
            TRACE(2 + a, sp_it, 4);
            // the next S first (it is what the softmax warps wait for), the stage releases after it
            if (more) issue_qk(kst, valid);
            if (j + 2 == n) tc_commit(bar_q_empty + 8 * a);
            tc_commit(bar_kv_empty + 8 * vst);
            if (s.nq == 2) {
              mbar_arrive(bar_mturn + 8 * (1 - a));
              ++mturn_it;
            }
            TRACE(2 + a, sp_it, 5);
            ++sp_it;
          } else {
            mbar_arrive(bar_kv_empty + 8 * vst);
            if (more) mbar_arrive(bar_kv_empty + 8 * kst);
          }
        }
        if (!ok) break;
        if (part) tc_commit(bar_o_final + 8 * a);
      }
    }
  } else {
    // ---------------------------------------------------------------- softmax warpgroups
    // Warps 0-3 own query tile 0, warps 4-7 query tile 1; a thread owns a row from the scores
    // to the output.  The groups never wait for each other.
    reg_alloc_softmax();
    const int a = warp >> 2;               // query tile of this warpgroup
    const int row = tid & 127;             // row inside the tile = TMEM lane
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const uint32_t t_S = t_lane + a * 128, t_O = t_lane + 256 + a * 128;
    const uint32_t my_p_full = bar_p_full + 8 * a;
    volatile int* my_flag = merge_flag + a;
    Sched sched(p, static_cast<int>(blockIdx.x));
    Seg s;
    uint32_t it = 0, seg_it = 0;
    bool ok = true;
    int seg_no = 0;
    CTRACE(1);
    // After a wait gave up (ok == false) a thread keeps walking its segments without working,
    // so that it still meets its group at the barrier of the next split-item epilogue, where
    // the whole group sees the abort flag and leaves together.
    while (sched.next(s)) {
      if (a >= s.nq) continue;             // a lone last query tile: nothing for group 1
      float m_run = -INFINITY, l_run = 0.f;
      const ValidKeys valid_of(p, s.b);
      for (int j = s.t0; j < s.t1 && ok; ++j) {
        const int valid = valid_of(j);
        TRACE(a, it, 0);
        ok = w.wait(bar_s_full + 8 * a, it & 1);
        if (!ok) break;
        tc_fence_after();
        if (it == 0) CTRACE(2);
        TRACE(a, it, 1);
        if (valid < kTileN)
          softmax_row_tile<true>(t_S, t_O, p.scale_log2e, valid, j == s.t0, m_run, l_run, my_p_full, a, it);
        else
          softmax_row_tile<false>(t_S, t_O, p.scale_log2e, kTileN, j == s.t0, m_run, l_run, my_p_full, a, it);
        ++it;
      }
      CTRACE(8 + seg_no);
      // ---- epilogue of this group's query tile ----
      if (ok) {
        ok = w.wait(bar_o_final + 8 * a, seg_it & 1);
        ++seg_it;
        tc_fence_after();
      }
      const int n = (2 * s.qp + a) * kTileM + row;
      uint4* const out_v = reinterpret_cast<uint4*>(out);
      const int64_t dst = ((static_cast<int64_t>(s.b) * p.L + n) * p.Hn + s.h) * (kHeadDim / 8);   // 16-byte vectors
      auto store_row = [&](int64_t d, const float* v, float inv_l) {   // 32 columns from vector d on
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint4 vv;
          vv.x = pack_bf16x2(v[8 * i + 0] * inv_l, v[8 * i + 1] * inv_l);
          vv.y = pack_bf16x2(v[8 * i + 2] * inv_l, v[8 * i + 3] * inv_l);
          vv.z = pack_bf16x2(v[8 * i + 4] * inv_l, v[8 * i + 5] * inv_l);
          vv.w = pack_bf16x2(v[8 * i + 6] * inv_l, v[8 * i + 7] * inv_l);
          UNSTEP_STORE(out_v, d + i, p.extent_out, vv, p.status);
        }
      };
      const bool whole = (s.t0 == 0 && s.t1 == s.tiles);
      if (whole) {
        // O / l -> bf16 -> out[b][n][h][:]: a thread writes its whole 256-byte row
        if (ok) {
          const float inv_l = 1.f / l_run;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            float o[32];
            tmem_ld32(t_O + q * 32, reinterpret_cast<uint32_t*>(o));
            tc_wait_ld32(reinterpret_cast<uint32_t*>(o));
            if (n < p.L) store_row(dst + 4 * q, o, inv_l);
          }
        }
      } else {
        // Part of a split item.  The parts of an item's query tile are merged by whichever of
        // them is done last, in part order (a fixed order, so the result does not depend on
        // which one that is); the merging part takes its own accumulator straight from TMEM.
        // A part that finds all others already published merges at once without publishing
        // itself; otherwise it publishes (O, m, l), counts itself in, and merges if that made
        // the count complete.
        const int c_lo = first_part_worker(p, s);
        const int c_hi = last_part_worker(p, s);
        const int others = c_hi - c_lo;
        int* counter = p.counters + 2 * s.item + a;
#ifdef UNSTEP_CHECK
        if (row == 0 && 2 * s.item + a >= p.extent_counters) atomicExch(p.status, static_cast<int>(UNSTEP_ERR_BOUNDS));
#endif
        if (row == 0 && ok) {
          int seen;
          asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
          *my_flag = (seen == others) ? 1 : 0;
        }
        group_barrier(a);
        if (*abort_flag) break;            // raised before the barrier by whoever gave up
        bool last = (*my_flag != 0);
        if (!last) {
          const int64_t mine = static_cast<int64_t>(2 * blockIdx.x + (s.first_in_worker ? 0 : 1)) * kPartFloats +
                               a * kPartTileFloats;   // first float of this part in the scratch
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint32_t o[32];
            tmem_ld32(t_O + q * 32, o);
            tc_wait_ld32(o);
#pragma unroll
            for (int i = 0; i < 32; ++i)
              UNSTEP_STORE(p.part, mine + (q * 32 + i) * 128 + row, p.extent_part, __uint_as_float(o[i]), p.status);
          }
          UNSTEP_STORE(p.part, mine + 128 * 128 + row, p.extent_part, m_run, p.status);
          UNSTEP_STORE(p.part, mine + 128 * 128 + 128 + row, p.extent_part, l_run, p.status);
          __threadfence();
          group_barrier(a);   // all of this part is published; everyone has read the flag
          if (row == 0) {
            // release: the group's stores (fenced above, ordered before this thread by the barrier)
            // become visible before the count; acquire: a merging part sees the other parts' stores
            __threadfence();
            const int before = atomicAdd(counter, 1);
            __threadfence();
            *my_flag = (before == others) ? 1 : 0;
          }
          group_barrier(a);
          last = (*my_flag != 0);
        }
        if (last) {
          __threadfence();   // acquire side for every thread that reads the other parts below
          if (row == 0) UNSTEP_STORE(p.counters, 2 * s.item + a, p.extent_counters, 0, p.status);   // ready for the next launch
          const int me = static_cast<int>(blockIdx.x);
          auto part_of = [&](int c) -> const float* {
            return p.part + (static_cast<int64_t>(2 * c + part_slot(p, c, s.item_step0)) * kPartFloats +
                             a * kPartTileFloats);
          };
          float m_all = m_run;
          for (int c = c_lo; c <= c_hi; ++c)
            if (c != me) m_all = fmaxf(m_all, __ldcg(part_of(c) + 128 * 128 + row));
          float l_sum = 0.f;
          for (int c = c_lo; c <= c_hi; ++c) {
            const float* pc = part_of(c);
            const float m_c = c == me ? m_run : __ldcg(pc + 128 * 128 + row);
            const float l_c = c == me ? l_run : __ldcg(pc + 128 * 128 + 128 + row);
            l_sum += l_c * ex2((m_c - m_all) * p.scale_log2e);
          }
          const float inv_l = 1.f / l_sum;
#pragma unroll 1
          for (int q = 0; q < 4; ++q) {   // 32 output columns at a time
            float acc[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) acc[i] = 0.f;
            for (int c = c_lo; c <= c_hi; ++c) {
              float v[32];
              float m_c;
              if (c == me) {
                tmem_ld32(t_O + 32 * q, reinterpret_cast<uint32_t*>(v));
                tc_wait_ld32(reinterpret_cast<uint32_t*>(v));
                m_c = m_run;
              } else {
                const float* pc = part_of(c);
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __ldcg(pc + (32 * q + i) * 128 + row);
                m_c = __ldcg(pc + 128 * 128 + row);
              }
              const float sc = ex2((m_c - m_all) * p.scale_log2e);
#pragma unroll
              for (int i = 0; i < 32; ++i) acc[i] = fmaf(v[i], sc, acc[i]);
            }
            if (n < p.L) store_row(dst + 4 * q, acc, inv_l);
          }
        }
      }
      tc_fence_before();
      CTRACE(3 + seg_no);
      ++seg_no;
    }
  }

  // ---- teardown: every role ends here, also after a timed-out wait --------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 10 && lane == 0 && *abort_flag) {
    // gave up: let copies that are still in flight land (bounded) before smem is released
    const long long t0 = clock64();
    while (clock64() - t0 < 4000000LL) {
    }
  }
  __syncthreads();
  if (warp == 8) tmem_dealloc(tmem_base, kTmemCols);
  CTRACE(7);
}

// A wait on a barrier that nothing ever arrives at, with a short limit: exercises the give-up
// path of Waiter (status word, flag, orderly return) without any other work.
__global__ void wait_limit_probe_kernel(long long limit_cycles) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  const Waiter w{&abort_flag, limit_cycles};
  w.wait(smem_u32(&bar), 0);
  __syncthreads();
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

struct DeviceInfo {
  bool ok = false;
  int sm_count = 0;
};

static const DeviceInfo& device_info() {
  static thread_local int cached_dev = -1;
  static thread_local DeviceInfo info;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    info.ok = false;
    return info;
  }
  if (dev != cached_dev) {
    info.ok = cudaDeviceGetAttribute(&info.sm_count, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
              cudaFuncSetAttribute(window_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   kAttnSmemBytes) == cudaSuccess;
    cached_dev = dev;
  }
  return info;
}

// Scratch for split items, one per (device, stream): calls on one stream run in order and may
// share it; calls on different streams may overlap on the GPU and must not.  Allocated on first
// use and kept; it only grows.
struct Workspace {
  float* part = nullptr;
  int* counters = nullptr;
  size_t slots = 0, n_counters = 0;
};
static std::mutex g_ws_mutex;
static std::map<std::pair<int, cudaStream_t>, Workspace> g_workspaces;

static int get_workspace(cudaStream_t st, size_t slots, size_t n_counters, Workspace* out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return UNSTEP_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_ws_mutex);
  Workspace& ws = g_workspaces[std::make_pair(dev, st)];
  if (ws.slots < slots) {
    if (ws.part != nullptr && cudaFree(ws.part) != cudaSuccess) return UNSTEP_ERR_CUDA;
    ws.part = nullptr;
    ws.slots = 0;
    if (cudaMalloc(&ws.part, slots * kPartFloats * sizeof(float)) != cudaSuccess) return UNSTEP_ERR_CUDA;
    ws.slots = slots;
  }
  if (ws.n_counters < n_counters) {
    if (ws.counters != nullptr && cudaFree(ws.counters) != cudaSuccess) return UNSTEP_ERR_CUDA;
    ws.counters = nullptr;
    ws.n_counters = 0;
    if (cudaMalloc(&ws.counters, n_counters * sizeof(int)) != cudaSuccess) return UNSTEP_ERR_CUDA;
    // cleared on the caller's stream, so that the clear is ordered before the kernel that follows
    // (a non-blocking stream is not ordered against the legacy default stream)
    if (cudaMemsetAsync(ws.counters, 0, n_counters * sizeof(int), st) != cudaSuccess) return UNSTEP_ERR_CUDA;
    ws.n_counters = n_counters;
  }
  *out = ws;
  return UNSTEP_OK;
}

// After a kernel gave up, arrival counters may be left non-zero: clear them all.
static void reset_workspace_counters() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return;
  std::lock_guard<std::mutex> lock(g_ws_mutex);
  for (auto& kv : g_workspaces)
    if (kv.first.first == dev && kv.second.counters != nullptr)
      cudaMemset(kv.second.counters, 0, kv.second.n_counters * sizeof(int));
}

// Device address of g_status on the current device, looked up once per device.
int* status_word() {
  static std::mutex mutex;
  static int* addr[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mutex);
  if (addr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_status) != cudaSuccess) return nullptr;
    addr[dev] = static_cast<int*>(ptr);
  }
  return addr[dev];
}

}  // namespace unstep

using namespace unstep;

// Hands out the scratch of one launch: `slots` partial-result slots and `n_counters` zeroed
// arrival counters.
typedef int (*ScratchFn)(cudaStream_t st, size_t slots, size_t n_counters, Workspace* out);   // an unstep_status

// Validation, work split, tensor maps and launch shared by the attention entry points.
// The cache has `sink_frames` slots in front of the ring (0 for the plain rolling window);
// stream b attends frames [0, min(sink_attend, lo)) and [lo, hi), lo = max(0, hi - window_frames).
static int window_attn_run(const unstep_shape_t* shape, const int32_t* start_frame,
                           int32_t window_frames, const void* q_rot, const void* ring_k,
                           const void* ring_v, void* out, void* cuda_stream, ScratchFn scratch,
                           int32_t sink_frames = 0, int32_t sink_attend = 0) {
  int rc = check_attn_args(shape, start_frame, window_frames, sink_frames, sink_attend);
  if (rc != UNSTEP_OK) return rc;
  const void* ptrs[] = {q_rot, ring_k, ring_v, out};
  for (const void* ptr : ptrs)
    if (ptr == nullptr || !aligned16(ptr)) return UNSTEP_ERR_INVALID_ARG;
  rc = check_device();
  if (rc != UNSTEP_OK) return rc;
  const DeviceInfo& info = device_info();
  if (!info.ok) return UNSTEP_ERR_CUDA;

  const uint64_t Hn = shape->heads;
  const uint64_t C = static_cast<uint64_t>(shape->ring_frames) + sink_frames;  // cache slots per stream
  const uint64_t T = static_cast<uint64_t>(shape->grid_h) * shape->grid_w;
  const uint64_t L = T * shape->chunk_frames;
  const uint64_t row_bytes = Hn * kHeadDim * 2;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

  AttnParams p;
  plan_shape(p, shape, sink_frames);
  for (int b0 = 0; b0 < shape->batch; b0 += kMaxStreamsPerLaunch) {
    const int nb = shape->batch - b0 < kMaxStreamsPerLaunch ? shape->batch - b0 : kMaxStreamsPerLaunch;
    rc = plan_launch(p, shape, start_frame + b0, nb, window_frames, sink_frames, sink_attend, info.sm_count);
    if (rc != UNSTEP_OK) return rc;
    Workspace ws;
    rc = scratch(st, 2 * static_cast<size_t>(p.n_workers), 2 * static_cast<size_t>(nb) * p.items_per_stream, &ws);
    if (rc != UNSTEP_OK) return rc;
    p.part = ws.part;
    p.counters = ws.counters;
    p.status = status_word();
    p.extent_out = static_cast<int64_t>(nb) * p.L * p.Hn * (kHeadDim / 8);
    p.extent_part = static_cast<int64_t>(ws.slots) * kPartFloats;
    p.extent_counters = static_cast<int64_t>(ws.n_counters);
    const char* qb = static_cast<const char*>(q_rot) + static_cast<uint64_t>(b0) * L * row_bytes;
    const char* kb = static_cast<const char*>(ring_k) + static_cast<uint64_t>(b0) * C * T * row_bytes;
    const char* vb = static_cast<const char*>(ring_v) + static_cast<uint64_t>(b0) * C * T * row_bytes;
    __nv_bfloat16* ob = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(out) +
                                                         static_cast<uint64_t>(b0) * L * row_bytes);
    CUtensorMap tm_q, tm_k, tm_v, tm_kf, tm_vf;
    const uint64_t qdims[4] = {kHeadDim, Hn, L, static_cast<uint64_t>(nb)};
    const uint64_t qstr[3] = {kHeadDim * 2, row_bytes, L * row_bytes};
    const uint64_t rdims[5] = {kHeadDim, Hn, T, C, static_cast<uint64_t>(nb)};
    const uint64_t rstr[4] = {kHeadDim * 2, row_bytes, T * row_bytes, C * T * row_bytes};
    const uint64_t fdims[4] = {kHeadDim, Hn, C * T, static_cast<uint64_t>(nb)};   // ring rows, flat
    const uint64_t fstr[3] = {kHeadDim * 2, row_bytes, C * T * row_bytes};
    if (!make_map(&tm_q, qb, 4, qdims, qstr, 2) || !make_map(&tm_k, kb, 5, rdims, rstr, 2) ||
        !make_map(&tm_v, vb, 5, rdims, rstr, 2) || !make_map(&tm_kf, kb, 4, fdims, fstr, 2) ||
        !make_map(&tm_vf, vb, 4, fdims, fstr, 2))
      return UNSTEP_ERR_CUDA;
    window_attn_kernel<<<p.n_workers, kThreads, kAttnSmemBytes, st>>>(tm_q, tm_k, tm_v, tm_kf, tm_vf, p, ob);
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) return UNSTEP_ERR_CUDA;
  }
  return UNSTEP_OK;
}

#ifdef UNSTEP_TRACE
extern "C" int unstep_debug_read_cta_trace(unsigned long long* host_out) {
  if (cudaDeviceSynchronize() != cudaSuccess) return UNSTEP_ERR_CUDA;
  return cudaMemcpyFromSymbol(host_out, g_cta_trace, sizeof(unsigned long long) * 160 * 16) == cudaSuccess
             ? UNSTEP_OK : UNSTEP_ERR_CUDA;
}
extern "C" int unstep_debug_read_trace(long long* host_out) {
  if (cudaDeviceSynchronize() != cudaSuccess) return UNSTEP_ERR_CUDA;
  return cudaMemcpyFromSymbol(host_out, g_trace, sizeof(long long) * 12 * 64 * 8) == cudaSuccess
             ? UNSTEP_OK : UNSTEP_ERR_CUDA;
}
#endif

extern "C" int unstep_window_attn(const unstep_shape_t* shape, const int32_t* start_frame,
                                  int32_t window_frames, const void* q_rot, const void* ring_k,
                                  const void* ring_v, void* out, void* cuda_stream) {
  return window_attn_run(shape, start_frame, window_frames, q_rot, ring_k, ring_v, out, cuda_stream,
                         get_workspace);
}

extern "C" int unstep_window_attn_sink(const unstep_shape_t* shape, int32_t sink_frames,
                                       const int32_t* start_frame, int32_t recent_frames,
                                       int32_t sink_attend, const void* q_rot, const void* cache_k,
                                       const void* cache_v, void* out, void* cuda_stream) {
  return window_attn_run(shape, start_frame, recent_frames, q_rot, cache_k, cache_v, out, cuda_stream,
                         get_workspace, sink_frames, sink_attend);
}

// --------------------------------------------------------------------------
// Attention without any allocation: the scratch is a fixed array in the library image.
// --------------------------------------------------------------------------
namespace unstep {

constexpr int kStaticMaxCtas = 148;                      // two partial-result slots per CTA
constexpr int kStaticMaxCounters = 2 * 32768;            // a pair of counters per work item
constexpr size_t kStaticCounterBytes = sizeof(int) * kStaticMaxCounters;
constexpr size_t kStaticScratchBytes =
    kStaticCounterBytes + sizeof(float) * 2 * kStaticMaxCtas * static_cast<size_t>(kPartFloats);

// Counters first, partial results after them.  In host code this name is only a handle for
// cudaGetSymbolAddress: it is not a device address and must never be passed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mutex;
static unsigned char* g_static_addr[kMaxDevices] = {};

// Device address of the array on the current device (looked up once per device).
static unsigned char* static_scratch_base() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_addr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return nullptr;
    g_static_addr[dev] = static_cast<unsigned char*>(ptr);
  }
  return g_static_addr[dev];
}

// Scratch source of the no-allocation entry point: carve the fixed array, clear the counters
// this launch will use (the array keeps the previous call's contents).
static int static_scratch(cudaStream_t st, size_t slots, size_t n_counters, Workspace* out) {
  if (slots > 2 * static_cast<size_t>(kStaticMaxCtas) || n_counters > static_cast<size_t>(kStaticMaxCounters))
    return UNSTEP_ERR_TOO_LARGE;
  unsigned char* base = static_scratch_base();
  if (base == nullptr) return UNSTEP_ERR_CUDA;
  if (cudaMemsetAsync(base, 0, n_counters * sizeof(int), st) != cudaSuccess) return UNSTEP_ERR_CUDA;
  out->counters = reinterpret_cast<int*>(base);
  out->part = reinterpret_cast<float*>(base + kStaticCounterBytes);
  out->slots = slots;
  out->n_counters = n_counters;
  return UNSTEP_OK;
}

}  // namespace unstep

extern "C" int unstep_window_attn_noalloc(const unstep_shape_t* shape, const int32_t* start_frame,
                                          int32_t window_frames, const void* q_rot, const void* ring_k,
                                          const void* ring_v, void* out, void* cuda_stream) {
  // size limits of the fixed array first, so that an oversized problem gets its own clear answer
  int rc = check_shape(shape, true);
  if (rc != UNSTEP_OK) return rc;
  const int64_t L = static_cast<int64_t>(shape->grid_h) * shape->grid_w * shape->chunk_frames;
  const int64_t q_pairs = ((L + kTileM - 1) / kTileM + 1) / 2;
  const int64_t streams = shape->batch < kMaxStreamsPerLaunch ? shape->batch : kMaxStreamsPerLaunch;
  if (2 * streams * shape->heads * q_pairs > kStaticMaxCounters) return UNSTEP_ERR_TOO_LARGE;
  rc = check_device();
  if (rc != UNSTEP_OK) return rc;
  const DeviceInfo& info = device_info();
  if (!info.ok) return UNSTEP_ERR_CUDA;
  if (info.sm_count > kStaticMaxCtas) return UNSTEP_ERR_TOO_LARGE;
  return window_attn_run(shape, start_frame, window_frames, q_rot, ring_k, ring_v, out, cuda_stream,
                         static_scratch);
}

extern "C" int unstep_attn_workers(int32_t* workers, int32_t* ctas_per_worker) {
  if (workers == nullptr || ctas_per_worker == nullptr) return UNSTEP_ERR_INVALID_ARG;
  const int rc = check_device();
  if (rc != UNSTEP_OK) return rc;
  const DeviceInfo& info = device_info();
  if (!info.ok) return UNSTEP_ERR_CUDA;
  *workers = info.sm_count;
  *ctas_per_worker = 1;
  return UNSTEP_OK;
}

#ifdef UNSTEP_CHECK
namespace unstep {
// One store just past the end of a 4-element buffer: a checking build must skip it and record it.
__global__ void check_probe_kernel(int* buf, int* status) {
  UNSTEP_STORE(buf, threadIdx.x, 4, 7, status);
}
}  // namespace unstep

extern "C" int unstep_selftest_bounds_check(int32_t* device_buf5, void* cuda_stream) {
  if (device_buf5 == nullptr) return UNSTEP_ERR_INVALID_ARG;
  const int rc = check_device();
  if (rc != UNSTEP_OK) return rc;
  int* st = status_word();
  if (st == nullptr) return UNSTEP_ERR_CUDA;
  check_probe_kernel<<<1, 5, 0, static_cast<cudaStream_t>(cuda_stream)>>>(device_buf5, st);
  g_launches.fetch_add(1);
  return cudaGetLastError() == cudaSuccess ? UNSTEP_OK : UNSTEP_ERR_CUDA;
}
#endif

extern "C" int unstep_selftest_wait_limit(int64_t limit_cycles, void* cuda_stream) {
  if (limit_cycles < 1 || limit_cycles > 4000000000LL) return UNSTEP_ERR_INVALID_ARG;
  const int rc = check_device();
  if (rc != UNSTEP_OK) return rc;
  wait_limit_probe_kernel<<<1, 64, 0, static_cast<cudaStream_t>(cuda_stream)>>>(limit_cycles);
  g_launches.fetch_add(1);
  return cudaGetLastError() == cudaSuccess ? UNSTEP_OK : UNSTEP_ERR_CUDA;
}

extern "C" void unstep_shutdown(void) {
  // frees the per-stream scratch buffers of every device; the next attention call makes new ones
  cudaDeviceSynchronize();
  int cur = 0;
  if (cudaGetDevice(&cur) != cudaSuccess) return;
  std::lock_guard<std::mutex> lock(g_ws_mutex);
  for (auto& kv : g_workspaces) {
    if (cudaSetDevice(kv.first.first) != cudaSuccess) continue;
    cudaDeviceSynchronize();
    if (kv.second.part != nullptr) cudaFree(kv.second.part);
    if (kv.second.counters != nullptr) cudaFree(kv.second.counters);
  }
  g_workspaces.clear();
  cudaSetDevice(cur);
}

extern "C" int unstep_poll_status(void) {
  if (cudaDeviceSynchronize() != cudaSuccess) return UNSTEP_ERR_CUDA;
  int st = 0, zero = 0;
  if (cudaMemcpyFromSymbol(&st, g_status, sizeof(int)) != cudaSuccess) return UNSTEP_ERR_CUDA;
  if (st != 0) {
    if (cudaMemcpyToSymbol(g_status, &zero, sizeof(int)) != cudaSuccess) return UNSTEP_ERR_CUDA;
    if (st == UNSTEP_ERR_TIMEOUT) reset_workspace_counters();
  }
  return st;
}
