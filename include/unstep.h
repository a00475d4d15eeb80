/*
 * unstep.h -- C ABI of the B200 (sm_100a) chunk-attention library.
 *
 * One self-attention layer of a chunk-causal video DiT, for one new latent chunk
 * (UnStep paper, Sec. "Increasing model efficiency" / "DiT runtime stack" and
 * appendix "Diffusion transformer runtime", appendix "KV attention window"):
 *
 *   1. unstep_rope_table      build the cached float32 cos/sin table of the chunk
 *   2. unstep_rope_kv_append  rotate Q and K, write K and V into the KV ring
 *   3. unstep_window_attn     attention of the chunk's queries over the window
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer unless the comment says HOST.
 *   - bf16 tensors are dense, row-major, 16-byte aligned; the caller owns all of
 *     them.  The only device memory the library creates is the scratch of
 *     unstep_window_attn (one buffer per stream, made on first use and kept).
 *   - All work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL
 *     is the legacy default stream).  No call synchronises or reads device data.
 *   - Return value: 0 on success, a negative unstep_status otherwise.  Arguments
 *     are validated before anything is launched; on error nothing was enqueued.
 *   - Chunk positions are plain host integers (the paper keeps the cache
 *     positions on the CPU so that no call needs a device-to-host read).
 *
 * Notation: B streams, Hn heads, D = 128, Fc chunk frames, T = grid_h*grid_w
 * tokens per latent frame, L = Fc*T queries per chunk, C ring capacity in
 * frames, token n = (f*grid_h + r)*grid_w + c.
 */
#ifndef UNSTEP_H_
#define UNSTEP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  UNSTEP_OK = 0,
  UNSTEP_ERR_INVALID_ARG = -1, /* null or misaligned pointer, bad size, bad window */
  UNSTEP_ERR_UNSUPPORTED = -2, /* head_dim != 128, device is not sm_100 */
  UNSTEP_ERR_CUDA = -3,        /* a CUDA runtime/driver call failed */
  UNSTEP_ERR_TIMEOUT = -4,     /* a bounded device-side wait expired (see unstep_poll_status) */
  UNSTEP_ERR_TOO_LARGE = -5,   /* the problem does not fit the fixed scratch of a no-allocation call */
  UNSTEP_ERR_BOUNDS = -6       /* checking build only: a kernel tried to store outside its buffer (see below) */
} unstep_status;

typedef struct {
  int32_t batch;        /* B: independent streams, each with its own ring */
  int32_t heads;        /* Hn */
  int32_t head_dim;     /* D, must be 128 */
  int32_t chunk_frames; /* Fc: latent frames per chunk */
  int32_t grid_h;       /* token rows per latent frame */
  int32_t grid_w;       /* token columns per latent frame; T = grid_h * grid_w */
  int32_t ring_frames;  /* C: capacity of the KV ring in latent frames */
  int32_t band_t;       /* head dims rotated by the frame position   (44) */
  int32_t band_h;       /* head dims rotated by the row position     (42) */
  int32_t band_w;       /* head dims rotated by the column position  (42) */
  double rope_base;     /* 10000.0 */
} unstep_shape_t;

/*
 * RoPE coefficient table of one chunk (appendix "Diffusion transformer runtime":
 * float32 sine and cosine tables, one coefficient vector per token, shared by all
 * heads, built once per starting latent frame index and grid size).
 *
 * Pair j in [0, 64) rotates (x[2j], x[2j+1]).  Pairs are split t | h | w in that
 * order, band_t/2, band_h/2, band_w/2 pairs; local pair i of a band of d_b dims has
 * omega = rope_base^(-2i/d_b); the angle is position * omega with the position
 * start_frame + f, r or c; angle and trig are evaluated in double and rounded once.
 *
 *   cos_out, sin_out : float32 [L, 64], written.
 *   start_frame      : absolute latent-frame index of the chunk's first frame, >= 0.
 * batch, heads and ring_frames of `shape` are not used by this call.
 */
int unstep_rope_table(const unstep_shape_t* shape, int32_t start_frame, float* cos_out,
                      float* sin_out, void* cuda_stream);

/*
 * Fused RoPE + KV-cache write (Sec. "DiT runtime stack": one kernel loads bf16,
 * rotates in float32, stores bf16; appendix: newly computed keys and values are
 * written at the chunk's cache position and repeated denoising calls overwrite the
 * same entries).
 *
 * For every stream b, token n, head h, pair j, with c = cos[n][j], s = sin[n][j]:
 *     y[2j]   = fl32(fl32(x[2j]*c) - fl32(x[2j+1]*s))
 *     y[2j+1] = fl32(fl32(x[2j]*s) + fl32(x[2j+1]*c))      (no fused multiply-add)
 * rounded to bf16 (nearest even).  q_out = rot(q_in); ring_k[b][slot][t] = rot(k_in),
 * ring_v[b][slot][t] = v_in (bit copy), slot = (start_frame[b] + f) mod C, where
 * n = f*T + t.  Slots of other frames are not touched.
 *
 *   start_frame : HOST int32 [B], each >= 0.
 *   q_in, k_in, v_in : bf16 [B, L, Hn, 128], read.
 *   cos, sin    : float32 [L, 64] per table; stream b uses the table at
 *                 cos + b*table_stream_stride (elements); stride 0 shares one table.
 *   q_out       : bf16 [B, L, Hn, 128], written; may be the same buffer as q_in.
 *   ring_k, ring_v : bf16 [B, C, T, Hn, 128], updated in place.
 */
int unstep_rope_kv_append(const unstep_shape_t* shape, const int32_t* start_frame,
                          const void* q_in, const void* k_in, const void* v_in, const float* cos,
                          const float* sin, int64_t table_stream_stride, void* q_out, void* ring_k,
                          void* ring_v, void* cuda_stream);

/*
 * Windowed attention of the chunk's queries (appendix "KV attention window": the
 * chunk attends the retained most recent latent frames, the current chunk included;
 * Sec. "DiT runtime stack": fixed-length attention, lengths taken from the call).
 *
 * Stream b attends the frames p in [max(0, start_frame[b] + Fc - window_frames),
 * start_frame[b] + Fc), all T tokens of each, read from ring slot p mod C.  No mask:
 *     out[b][n][h] = softmax_m( q_rot[b][n][h] . k_m / sqrt(128) ) v_m
 * bf16 operands, float32 accumulation, bf16 result.
 *
 *   start_frame   : HOST int32 [B], each >= 0.
 *   window_frames : Fc <= window_frames <= C.
 *   q_rot         : bf16 [B, L, Hn, 128], the q_out of unstep_rope_kv_append.
 *   ring_k, ring_v: bf16 [B, C, T, Hn, 128], read.  Every attended frame must have
 *                   been appended and not yet overwritten (true when chunks arrive in
 *                   order and window_frames <= C).
 *   out           : bf16 [B, L, Hn, 128], written.
 * Scratch: work items that are split across thread blocks exchange partial results through a
 * buffer the library keeps per (device, stream).  The first call on a stream creates it with
 * cudaMalloc (about 40 MB): make that call outside any stream capture.  Calls on one stream
 * share the buffer safely; calls on different streams use different buffers.  A buffer is replaced
 * by a larger one when a later call on its stream needs more (more SMs or more work items).
 * CUDA graphs: a call captured into a graph freezes the addresses of the capture stream's buffer
 * into the graph.  Such a graph is invalid after unstep_shutdown() and after a larger problem was
 * run on the capture stream (both free the buffer), and its replays must not overlap on the GPU
 * with each other or with direct calls on the capture stream.  Capture all graphs that may replay
 * back to back on one stream, after one uncaptured call of the largest problem on that stream.
 */
int unstep_window_attn(const unstep_shape_t* shape, const int32_t* start_frame,
                       int32_t window_frames, const void* q_rot, const void* ring_k,
                       const void* ring_v, void* out, void* cuda_stream);

/*
 * Sink + sliding window (Sec. "Limited KV attention window", appendix "KV attention window":
 * the first 3 latent frames are kept as sink frames and never evicted, the 6 most recent
 * frames, the current chunk included, form the sliding window; selected layers attend 2 sink
 * frames and the same 6 recent frames).
 *
 * The cache of a stream has sink_frames slots in front of the ring:
 *     cache_k, cache_v : bf16 [B, sink_frames + C, T, Hn, 128]
 *     frame p lives in slot p                              if p <  sink_frames
 *                      slot sink_frames + (p - sink_frames) mod C   otherwise.
 * unstep_rope_kv_append_sink is unstep_rope_kv_append with that slot rule.
 * unstep_window_attn_sink attends, for stream b with hi = start_frame[b] + Fc and
 * lo = max(0, hi - recent_frames), the frames [0, min(sink_attend, lo)) and [lo, hi): while the
 * recent part still reaches the sink this is every frame so far, afterwards sink + recent.
 *   sink_frames  : >= 0; 0 makes both calls identical to the plain ones.
 *   recent_frames: Fc <= recent_frames <= C.     sink_attend: 0 <= sink_attend <= sink_frames.
 * All other arguments as in unstep_rope_kv_append / unstep_window_attn.
 */
int unstep_rope_kv_append_sink(const unstep_shape_t* shape, int32_t sink_frames,
                               const int32_t* start_frame, const void* q_in, const void* k_in,
                               const void* v_in, const float* cos, const float* sin,
                               int64_t table_stream_stride, void* q_out, void* cache_k, void* cache_v,
                               void* cuda_stream);
int unstep_window_attn_sink(const unstep_shape_t* shape, int32_t sink_frames,
                            const int32_t* start_frame, int32_t recent_frames, int32_t sink_attend,
                            const void* q_rot, const void* cache_k, const void* cache_v, void* out,
                            void* cuda_stream);

/*
 * RMS normalisation of q and k fused in front of the rotation (appendix "Diffusion transformer
 * runtime": q and k are normalised before they are split into heads; the paper gives no formula,
 * this is the textbook RMSNorm over the whole token vector of Hn*128 channels with a learned gain):
 *     y = x / sqrt(mean(x^2) + eps) * gain,   rounded to bf16, then rotated and appended exactly
 * as unstep_rope_kv_append_sink does (v is copied, not normalised).  The mean of squares is
 * accumulated in double and rounded to float32; sqrt, reciprocal and the two products are single
 * float32 operations.  Saves one read and one write of q and k compared with a separate norm.
 *   gain_q, gain_k : float32 [Hn*128], read.     eps : >= 0.
 *   sink_frames    : 0 for the plain ring.  All other arguments as in unstep_rope_kv_append_sink.
 */
int unstep_rmsnorm_rope_kv_append(const unstep_shape_t* shape, int32_t sink_frames,
                                  const int32_t* start_frame, const void* q_in, const void* k_in,
                                  const void* v_in, const float* gain_q, const float* gain_k, float eps,
                                  const float* cos, const float* sin, int64_t table_stream_stride,
                                  void* q_out, void* cache_k, void* cache_v, void* cuda_stream);

/*
 * unstep_window_attn for callers that must not allocate.  (The paper has no counterpart:
 * this is a deployment variant of the call above, same arguments, same result.)
 *
 * unstep_window_attn keeps a scratch buffer per stream and creates it with cudaMalloc the first
 * time it is needed.  That is not acceptable everywhere: a serving process whose device memory
 * has been handed over in full to a framework's caching allocator has nothing left for a raw
 * cudaMalloc to return; a latency-critical loop cannot take the device-wide synchronisation an
 * allocation may imply; and some deployments forbid any allocation after start-up so that the
 * memory footprint is known before the first request.  This entry point calls no cudaMalloc,
 * cudaFree or any other allocating routine.  Its scratch is a fixed array that is part of the
 * library image: about 39.8 MB of device memory on every GPU that loads the library, held
 * until the process exits, whether or not this call is ever used.
 *
 * Limits (beyond them the call returns UNSTEP_ERR_TOO_LARGE and launches nothing):
 *   - at most 148 SMs on the device (the array has two partial-result slots per SM);
 *   - min(batch, 32) * heads * ceil(ceil(L / 128) / 2) <= 32768 (one pair of arrival counters
 *     per work item of a launch).
 *
 * Set-up: the first call on each device looks up the device address of the array, with that
 * device current, and remembers it.  Make that first call outside any stream capture.
 *
 * Sharing: every call on a device uses the same array, and the array keeps whatever the last
 * call left in it.  Each call clears the counters it needs (stream-ordered, on cuda_stream)
 * before its kernel runs.  Calls that can overlap on the GPU (different streams, or several
 * host threads) race on the array and corrupt each other's results: serialise them, or use
 * unstep_window_attn, which keeps one scratch per stream.
 */
int unstep_window_attn_noalloc(const unstep_shape_t* shape, const int32_t* start_frame,
                               int32_t window_frames, const void* q_rot, const void* ring_k,
                               const void* ring_v, void* out, void* cuda_stream);

/*
 * The work split of one unstep_window_attn(_sink) launch, listed on the host by the same integer
 * code that the kernel's roles run on the device (the paper has no counterpart: a diagnostic for
 * tests and tuning).  No device is touched and no GPU is needed.
 *
 * The launch is cut into work items (stream, head, pair of 128-query tiles); an item has one step
 * per 128-key tile of its window.  Each of at most `max_workers` workers (one per SM) first takes
 * whole items round-robin; what is left over is one sequence of steps cut into equal contiguous
 * shares, so an item there may be split along its keys into parts that different workers compute
 * and the last one to finish merges.
 *
 *   segs     : HOST int32 [max_segs][10], written (may be NULL when max_segs is 0).  One row per
 *              segment in the order the worker walks them: worker, stream, head, query pair,
 *              query tiles in the pair (1 or 2), first key tile, end key tile (exclusive), key
 *              tiles of the whole item, number of parts the item is split into (1 = whole), and the
 *              scratch slot (0 or 1) the part is published in (-1 for a whole item).
 *   n_segs   : HOST int32, written: the number of segments of the launch (may exceed max_segs; only
 *              the first max_segs rows are written).
 * Only the first launch of the call is listed (the first 32 streams).  Arguments are checked as in
 * unstep_window_attn_sink; sink_frames = 0 lists the plain rolling window.
 */
int unstep_window_attn_plan(const unstep_shape_t* shape, int32_t sink_frames, const int32_t* start_frame,
                            int32_t recent_frames, int32_t sink_attend, int32_t max_workers,
                            int32_t* segs, int32_t max_segs, int32_t* n_segs);

/*
 * How the attention calls will use the current device (the paper has no counterpart): the number
 * of workers of a full-size launch (the `max_workers` to give unstep_window_attn_plan: one per SM)
 * and the thread blocks per worker (1: every worker is one persistent thread block).
 *   workers, ctas_per_worker : HOST int32, written.
 */
int unstep_attn_workers(int32_t* workers, int32_t* ctas_per_worker);

/* Static, human-readable text for a status code. */
const char* unstep_strerror(int code);

/*
 * Device status word of the current device: 0, or UNSTEP_ERR_TIMEOUT if a kernel gave
 * up on a bounded wait since the last poll (the word is cleared by the poll).  This
 * call synchronises the device; it is a diagnostic, not part of the hot path.
 * In a checking build (the library compiled with -DUNSTEP_CHECK, slower) every global store of
 * the kernels is tested against the extent of the buffer it belongs to; a store outside is
 * skipped, never made, and the poll returns UNSTEP_ERR_BOUNDS.  Nothing traps.
 */
int unstep_poll_status(void);

/*
 * Self-test of the bounded device-side waits: launches one small kernel that waits, with the same
 * code the attention kernel uses, on a barrier that nothing signals, gives up after `limit_cycles`
 * SM clock cycles (1 .. 4e9), records UNSTEP_ERR_TIMEOUT in the status word and returns normally.
 * Nothing traps or hangs; the context stays usable.  Afterwards unstep_poll_status() returns
 * UNSTEP_ERR_TIMEOUT once.
 */
int unstep_selftest_wait_limit(int64_t limit_cycles, void* cuda_stream);

/*
 * Optional: waits for the devices to go idle and frees the scratch buffers unstep_window_attn
 * created (all devices, all streams).  The library stays usable; the next call makes new ones.
 */
void unstep_shutdown(void);

/* Number of kernels the library has launched in this process (all devices). */
int64_t unstep_launch_count(void);

#ifdef UNSTEP_CHECK
/*
 * Only in a checking build: launches one kernel whose fifth thread stores one element past the
 * end of a 4-element range of `device_buf5` (DEVICE int32 [5]).  The store is skipped, the first
 * four elements become 7, element 4 keeps its value and unstep_poll_status() then returns
 * UNSTEP_ERR_BOUNDS once.  Shows that the checks are armed; nothing faults.
 */
int unstep_selftest_bounds_check(int32_t* device_buf5, void* cuda_stream);
#endif

#ifdef UNSTEP_TRACE
/*
 * Only in a library built with -DUNSTEP_TRACE (a diagnostic build, slower): the attention kernel
 * stamps the clock at the hand-overs between its roles.  Both calls synchronise the device and
 * copy the stamps of the last launch to HOST memory: [12 roles][64 key tiles][8 events] clock64
 * values of thread block 0, and [160 thread blocks][16 events] global-timer values.
 */
int unstep_debug_read_trace(long long* host_out);
int unstep_debug_read_cta_trace(unsigned long long* host_out);
#endif

#ifdef __cplusplus
}
#endif
#endif /* UNSTEP_H_ */
