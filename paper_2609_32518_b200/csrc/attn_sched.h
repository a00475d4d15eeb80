// Work split of the windowed attention: which key tiles of which (stream, head, query-tile pair)
// each worker (a CTA, or a CTA pair) processes, and how the parts of an item that is split along
// its keys find each other.  Pure integer arithmetic, compiled for the host (launch set-up, the
// plan entry point and its CPU tests) and for the device (every role of the kernel walks the same
// sequence).
#pragma once

#include <stdint.h>

#include "common.h"

#if defined(__CUDACC__)
#define UNSTEP_HD __host__ __device__ __forceinline__
#else
#define UNSTEP_HD inline
#endif

namespace unstep {

constexpr int kTileM = 128;                 // queries per tile (two tiles per work item)
constexpr int kTileN = 128;                 // keys per tile
constexpr int kMinStepsPerWorker = 4;       // a launch smaller than this per worker uses fewer workers

struct AttnParams {
  int32_t Hn, L, T, C;
  int32_t q_tiles;          // ceil(L / 128)
  int32_t q_pairs;          // ceil(q_tiles / 2)
  int32_t tiles_per_frame;  // ceil(T / 128)
  int32_t flat;             // 1: key tiles run across frame boundaries inside a slot run
  int32_t n_streams;
  float scale_log2e;        // log2(e) / sqrt(128)
  int32_t items_per_stream; // Hn * q_pairs
  int32_t n_workers;        // workers of the launch (grid size, or clusters)
  int32_t n_active;         // workers that take a share of the remainder: min(n_workers, steps / 4), >= 1
  int32_t full_rounds;      // whole rounds per stream: items_per_stream / n_workers
  int64_t total_steps;      // remainder: sum over the leftover items of their key tiles
  float* part;              // workspace: partial results of split items, kPartFloats per slot
  int* counters;            // workspace: arrivals per (item, query tile), zero between launches
  int* status;              // status word; with the extents below, for checking builds
  int64_t extent_out;       // 16-byte vectors of `out` that belong to this launch's streams
  int64_t extent_part;      // floats of `part`
  int64_t extent_counters;  // ints of `counters`
  int32_t sink;             // S: cache slots [0, S) hold frames [0, S) for good, the ring follows
  int32_t first_frame[kMaxStreamsPerLaunch];  // first frame of the recent part of stream b
  int32_t n_sink[kMaxStreamsPerLaunch];       // sink frames attended in front of the recent part
  int32_t tiles[kMaxStreamsPerLaunch];        // key tiles of one item of stream b
  // flat mode: the attended frames are at most three runs of consecutive cache slots (sink
  // prefix, ring up to its end, ring from its start); run r starts at cache row run_row0 and
  // has run_rows keys, its tiles are [run_tile_end[r-1], run_tile_end[r])
  int32_t run_row0[kMaxStreamsPerLaunch][3];
  int32_t run_rows[kMaxStreamsPerLaunch][3];
  int32_t run_tile_end[kMaxStreamsPerLaunch][3];
  int64_t step_base[kMaxStreamsPerLaunch];    // remainder steps of all streams before b
};

// One unit of work of a worker: key tiles [t0, t1) of item (b, h, query-tile pair qp).
struct Seg {
  int b, h, qp, nq, t0, t1;
  int tiles;             // key tiles of the whole item
  int item;              // item index inside the launch
  int64_t item_step0;    // global step index of the item's first tile
  bool first_in_worker;  // this segment starts the worker's range
};

// Where key tile j of an item of stream b lives and how many of its 128 keys are real.
// Flat mode: tiles are cut from the runs of consecutive ring slots, so only the last tile of
// a run is ragged; it is fetched through the per-frame map, whose zero fill ends it cleanly at
// the end of its frame (a run ends on a frame end, and the ragged tile is shorter than a frame).
// Per-frame mode (frames shorter than a tile): every tile lies inside one frame.
struct TileInfo {
  int valid;      // real keys in the tile, 1..128
  bool framed;    // fetch through the (token, slot) map at (tok0, slot), else the flat map at row
  int row, slot, tok0;
};
UNSTEP_HD TileInfo tile_info(const AttnParams& p, int b, int j) {
  TileInfo t;
  if (p.flat) {
    int r = 0;
    if (j >= p.run_tile_end[b][0]) r = (j >= p.run_tile_end[b][1]) ? 2 : 1;
    const int t_begin = r == 0 ? 0 : p.run_tile_end[b][r - 1];
    const int tt = j - t_begin;
    const int rows = p.run_rows[b][r];
    const int row0 = p.run_row0[b][r];
    const int ntl = p.run_tile_end[b][r] - t_begin;
    const bool last = (tt == ntl - 1);
    t.valid = last ? rows - kTileN * tt : kTileN;
    t.framed = last;
    t.row = row0 + kTileN * tt;
    t.slot = (row0 + rows - 1) / p.T;
    t.tok0 = p.T - t.valid;
  } else {
    const int fi = j / p.tiles_per_frame;
    const int tt = j - fi * p.tiles_per_frame;
    t.valid = (tt == p.tiles_per_frame - 1) ? p.T - kTileN * tt : kTileN;
    t.framed = true;
    t.row = 0;
    // frame list = the attended sink frames, then the recent frames
    const int frame = fi < p.n_sink[b] ? fi : p.first_frame[b] + fi - p.n_sink[b];
    t.slot = frame < p.sink ? frame : p.sink + (frame - p.sink) % p.C;
    t.tok0 = kTileN * tt;
  }
  return t;
}

// Work split.  Items are ordered stream, head, query pair, so neighbouring workers work on the
// same head and share its K/V through L2.
//   1. Whole rounds: while a stream still has at least n_workers items, worker c takes item
//      (round * n_workers + c) whole.  All workers walk the key tiles in step, so a K/V tile is
//      fetched from HBM once and then hit in L2 by the other workers of the head.
//   2. Remainder: the leftover items of all streams (fewer than n_workers per stream) form one
//      sequence of (item, key tile) steps, and each of the first n_active workers takes an equal
//      contiguous share of it (n_active <= total_steps, so no share is empty and the workers
//      that hold parts of an item are exactly those between the owners of its first and last
//      step).  An item that straddles a boundary is split along its keys; the parts are merged
//      by whichever worker finishes last.
struct Sched {
  int64_t lo, hi, cur;
  int b_round, round;   // position in the whole rounds
  int me;
  const AttnParams& p;
  UNSTEP_HD static int64_t worker_lo(const AttnParams& p, int64_t c) {
    return c >= p.n_active ? p.total_steps : p.total_steps * c / p.n_active;
  }
  UNSTEP_HD static int worker_of(const AttnParams& p, int64_t step) {
    int64_t c = step * p.n_active / p.total_steps;
    while (c + 1 < p.n_active && worker_lo(p, c + 1) <= step) ++c;
    while (c > 0 && worker_lo(p, c) > step) --c;
    return static_cast<int>(c);
  }
  UNSTEP_HD Sched(const AttnParams& prm, int worker) : me(worker), p(prm) {
    lo = worker_lo(p, worker);
    hi = worker_lo(p, worker + 1);
    cur = lo;
    b_round = 0;
    round = 0;
  }
  UNSTEP_HD void decode(Seg& s, int b, int in_stream) const {
    s.b = b;
    s.tiles = p.tiles[b];
    s.item = b * p.items_per_stream + in_stream;
    s.qp = in_stream % p.q_pairs;
    s.h = in_stream / p.q_pairs;
    s.nq = (2 * s.qp + 1 < p.q_tiles) ? 2 : 1;
  }
  UNSTEP_HD bool next(Seg& s) {
    while (b_round < p.n_streams) {          // whole rounds
      if (round < p.full_rounds) {
        decode(s, b_round, round * p.n_workers + me);
        s.t0 = 0;
        s.t1 = s.tiles;
        s.item_step0 = 0;
        s.first_in_worker = false;
        ++round;
        return true;
      }
      round = 0;
      ++b_round;
    }
    if (cur >= hi) return false;             // remainder
    int b = 0;
    while (b + 1 < p.n_streams && p.step_base[b + 1] <= cur) ++b;
    const int tiles = p.tiles[b];
    const int64_t rel = cur - p.step_base[b];
    const int left_item = static_cast<int>(rel / tiles);
    decode(s, b, p.full_rounds * p.n_workers + left_item);
    s.t0 = static_cast<int>(rel - static_cast<int64_t>(left_item) * tiles);
    const int64_t left = hi - cur;
    s.t1 = (left < tiles - s.t0) ? s.t0 + static_cast<int>(left) : tiles;
    s.item_step0 = cur - s.t0;
    s.first_in_worker = (cur == lo);
    cur += s.t1 - s.t0;
    return true;
  }
};

// Parts of a split item: the workers that own its first and its last step, and the scratch slot
// (0 or 1 of the two a worker has) in which worker c publishes its part of the item that starts
// at global step item_step0.
UNSTEP_HD int first_part_worker(const AttnParams& p, const Seg& s) { return Sched::worker_of(p, s.item_step0); }
UNSTEP_HD int last_part_worker(const AttnParams& p, const Seg& s) {
  return Sched::worker_of(p, s.item_step0 + s.tiles - 1);
}
UNSTEP_HD int part_slot(const AttnParams& p, int c, int64_t item_step0) {
  return Sched::worker_lo(p, c) >= item_step0 ? 0 : 1;   // 0: the part starts the worker's range
}

// Fills the per-launch part of `p` for streams [b0, b0 + nb): the attended frames of each stream
// cut into runs of consecutive cache slots, the key tiles, and the split of the work over at
// most `max_workers` workers.  The shape-wide fields (Hn, L, T, C, q_tiles, q_pairs,
// tiles_per_frame, flat, items_per_stream, sink) must already be set.  Host only.
inline int plan_launch(AttnParams& p, const unstep_shape_t* shape, const int32_t* start_frame, int nb,
                       int32_t window_frames, int32_t sink_frames, int32_t sink_attend, int max_workers) {
  p.n_streams = nb;
  for (int i = 0; i < nb; ++i) {
    const int hi = start_frame[i] + shape->chunk_frames;
    const int lo = hi - window_frames > 0 ? hi - window_frames : 0;
    const int n_sink = sink_attend < lo ? sink_attend : lo;   // sink frames not already in the recent part
    p.first_frame[i] = lo;
    p.n_sink[i] = n_sink;
    for (int r = 0; r < 3; ++r) p.run_row0[i][r] = p.run_rows[i][r] = p.run_tile_end[i][r] = 0;
    if (p.flat) {
      // walk the attended frames in order and cut them into runs of consecutive cache slots
      int n_runs = 0, prev_slot = -2;
      for (int k = 0; k < n_sink + hi - lo; ++k) {
        const int frame = k < n_sink ? k : lo + k - n_sink;
        const int slot = frame < sink_frames ? frame : sink_frames + (frame - sink_frames) % shape->ring_frames;
        if (slot != prev_slot + 1) {
          if (n_runs == 3) return UNSTEP_ERR_INVALID_ARG;  // cannot happen: sink, ring end, ring start
          p.run_row0[i][n_runs++] = slot * p.T;
        }
        p.run_rows[i][n_runs - 1] += p.T;
        prev_slot = slot;
      }
      int tiles = 0;
      for (int r = 0; r < 3; ++r) {
        tiles += (p.run_rows[i][r] + kTileN - 1) / kTileN;
        p.run_tile_end[i][r] = tiles;
      }
      p.tiles[i] = tiles;
    } else {
      p.tiles[i] = (n_sink + hi - lo) * p.tiles_per_frame;
    }
  }
  // one worker per SM (or SM pair), fewer when the whole launch is small
  int64_t all_steps = 0;
  for (int i = 0; i < nb; ++i) all_steps += static_cast<int64_t>(p.items_per_stream) * p.tiles[i];
  int64_t want = all_steps / kMinStepsPerWorker;
  if (want < 1) want = 1;
  p.n_workers = static_cast<int32_t>(want < max_workers ? want : max_workers);
  p.full_rounds = p.items_per_stream / p.n_workers;
  const int leftover = p.items_per_stream - p.full_rounds * p.n_workers;
  int64_t steps = 0;
  for (int i = 0; i < nb; ++i) {
    p.step_base[i] = steps;
    steps += static_cast<int64_t>(leftover) * p.tiles[i];
  }
  p.total_steps = steps;
  int64_t active = steps / kMinStepsPerWorker;
  if (active < 1) active = 1;
  p.n_active = static_cast<int32_t>(active < p.n_workers ? active : p.n_workers);
  return UNSTEP_OK;
}

// Shape-wide fields of the parameter block.
inline void plan_shape(AttnParams& p, const unstep_shape_t* shape, int32_t sink_frames) {
  const int64_t T = static_cast<int64_t>(shape->grid_h) * shape->grid_w;
  const int64_t L = T * shape->chunk_frames;
  p.sink = sink_frames;
  p.Hn = shape->heads;
  p.L = static_cast<int32_t>(L);
  p.T = static_cast<int32_t>(T);
  p.C = shape->ring_frames;
  p.q_tiles = static_cast<int32_t>((L + kTileM - 1) / kTileM);
  p.q_pairs = (p.q_tiles + 1) / 2;
  p.tiles_per_frame = static_cast<int32_t>((T + kTileN - 1) / kTileN);
  p.flat = (T >= kTileN) ? 1 : 0;  // a ragged tile must fit inside one frame
  p.scale_log2e = 1.4426950408889634f / 11.313708498984761f;   // log2(e) / sqrt(128)
  p.items_per_stream = p.Hn * p.q_pairs;
  p.part = nullptr;
  p.counters = nullptr;
  p.status = nullptr;
  p.extent_out = p.extent_part = p.extent_counters = 0;
}

// Argument checks shared by the attention entry points and the plan entry point (no device needed).
inline int check_attn_args(const unstep_shape_t* shape, const int32_t* start_frame, int32_t window_frames,
                           int32_t sink_frames, int32_t sink_attend) {
  const int rc = check_shape(shape, true);
  if (rc != UNSTEP_OK) return rc;
  if (start_frame == nullptr) return UNSTEP_ERR_INVALID_ARG;
  if (window_frames < shape->chunk_frames || window_frames > shape->ring_frames) return UNSTEP_ERR_INVALID_ARG;
  if (sink_frames < 0 || sink_frames > 4096 || sink_attend < 0 || sink_attend > sink_frames)
    return UNSTEP_ERR_INVALID_ARG;
  for (int b = 0; b < shape->batch; ++b)
    if (start_frame[b] < 0 || start_frame[b] > INT32_MAX - shape->chunk_frames) return UNSTEP_ERR_INVALID_ARG;
  const uint64_t C = static_cast<uint64_t>(shape->ring_frames) + sink_frames;
  const uint64_t T = static_cast<uint64_t>(shape->grid_h) * shape->grid_w;
  if (C * T >= (uint64_t(1) << 30)) return UNSTEP_ERR_INVALID_ARG;  // cache rows are 32-bit coordinates
  return UNSTEP_OK;
}

}  // namespace unstep
