/*
 * dgs.h -- C ABI of the DGS push / apply / pull loop on one GPU.
 *
 * DGS (dual-way gradient sparsification with sparsification-aware momentum,
 * arXiv 1910.10929) lets N asynchronous workers exchange sparse updates with a
 * parameter server in both directions.  This library keeps the N workers and the
 * server on ONE device and runs, per arrival ("event") of a worker k:
 *
 *   push   worker side, Algorithm 3:  t = m*u_k + eta*grad;  per layer keep the
 *          k_j entries of largest |t| (the packet g);  u_k <- t on the sent
 *          entries and t*(1/m) on the others (Eq. 11a, Eq. 12).
 *   apply  server side, Algorithm 2:  M <- M - decode(g)  (Eq. 1).  The model is
 *          stored as theta = theta_0 + M (Eq. 2) and every worker's model
 *          difference D_q = M - v_q (Eq. 3) moves with M.
 *   pull   server side, Algorithm 2 with secondary compression (Eq. 6a/6b):
 *          per layer keep the k_j entries of largest |D_k| (the packet G), clear
 *          them in D_k (v_k <- v_k + G), leave the rest as the server's residual;
 *          optionally the worker installs theta_k <- theta_k + G (Eq. 5).
 *
 * Conventions
 *   - All numbers are IEEE binary32; every arithmetic step is one rounded
 *     operation (no fused multiply-add, no flush-to-zero), so results do not
 *     depend on launch shapes.  Inputs must be finite.
 *   - "Largest |x|" compares the bit pattern of x with the sign bit cleared.
 *     Exactly k_j entries are kept per layer; among equal magnitudes the lowest
 *     index wins.  Packets list (index, value) pairs in ascending index order.
 *   - DEVICE pointers are marked DEVICE, everything else is host memory.
 *   - The caller owns all device memory (the arena); the library allocates no device
 *     memory.  Calls only enqueue work and return.  The work runs on streams of the
 *     library's own (several for the pushes, one for the apply, several for the pulls, so
 *     that the push of the next events overlaps the server side of the current one; a
 *     dependency tracker keeps, per buffer, the order of the calls); it is ordered after
 *     everything the caller had enqueued on the stream given at dgs_init when the call
 *     was made.  Results (packets, state) are complete for that stream after dgs_flush,
 *     and for the host after any call that is documented to wait.  One host thread per
 *     context.
 *   - The library's streams are eleven (four for pushes, one for the apply, six for pulls).
 *     The CUDA driver maps streams onto a fixed number of hardware queues, 8 unless the
 *     environment variable CUDA_DEVICE_MAX_CONNECTIONS says otherwise, and streams that
 *     share a queue run one after the other.  The variable is read when the process creates
 *     its CUDA context, so a process that wants the overlap must set it (to 12 or more; 32
 *     is the most) BEFORE its first CUDA call; the library cannot do it later.  Results do
 *     not depend on it, only speed does.  dgs_hardware_queues tells what the process has.
 *   - 16-bit packet values (DGS_PACKET_BF16 / DGS_PACKET_FP16; not part of the paper's algorithms, its
 *     closing section names the combination with other compression as the next step): the selection is
 *     made on the unrounded magnitudes; a packet carries q = the selected value rounded to the 16-bit
 *     format (nearest, ties to even), stored as the float32 number with that value, so that a transport
 *     may ship 16 bits per value.  A push leaves the worker's velocity as Eq. 12 says (a sent entry keeps
 *     t; sparsification-aware momentum has no residual that could take t - q); under DGS_RESIDUAL_MODE
 *     the residual keeps t - q.  A pull lowers D_k by q (Eq. 6b: v_k <- v_k + G with the G that was
 *     sent), so what rounding left behind stays with the server and goes out with a later pull.
 *   - Every function returns DGS_OK (0) or a negative dgs_error.  Nothing aborts,
 *     throws or waits without bound.
 */
#ifndef DGS_H_
#define DGS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DGS_OK = 0,
  DGS_EINVAL = -1,   /* null pointer, worker out of range, bad segment table, m not in (0,1], n >= 2^32, misaligned pointer */
  DGS_ENOMEM = -2,   /* arena too small */
  DGS_ECUDA = -3,    /* a CUDA runtime call or launch failed; see dgs_last_cuda_error */
  DGS_ETIMEOUT = -4, /* a bounded device-side wait gave up (reported by dgs_status) */
  DGS_ESTATE = -5,   /* context already freed or unusable after an earlier error */
  DGS_ELIMIT = -6    /* size beyond a fixed capacity: dgs_topk_encode_static, or (as device status) more nonzero
                        entries than a dgs_worker_pull_all packet can carry */
} dgs_error;

typedef struct dgs_ctx dgs_ctx; /* opaque, host side */

/* One layer j of the per-layer loops of Algorithm 3 / Algorithm 2: a contiguous
 * slice [offset, offset+len) of the flat parameter vector that is sparsified on
 * its own.  Segments must be listed in ascending order and tile [0, n) exactly.
 * 1 <= k_push <= len and 1 <= k_pull <= len. */
typedef struct {
  uint64_t offset;
  uint64_t len;
  uint32_t k_push; /* entries the worker sends per push from this layer   */
  uint32_t k_pull; /* entries the server sends per pull from this layer   */
} dgs_segment;

/* A sparse update in coordinate format (the paper's encode()): count pairs,
 * idx ascending.  Packets returned by the library point into the context's own
 * packet slots (DEVICE) and stay valid until the next call that produces a packet
 * of the same kind (push or pull). */
typedef struct {
  const uint32_t* idx; /* DEVICE u32[count], flat parameter index */
  const float* val;    /* DEVICE f32[count]                        */
  uint32_t count;      /* = sum of k_push (push) or k_pull (pull)  */
} dgs_packet;

/* A sparse update whose number of entries is only known on the device (the pull without
 * secondary compression sends however many entries the difference vector holds). */
typedef struct {
  const uint32_t* idx;   /* DEVICE u32[capacity], ascending; the first *count entries are valid */
  const float* val;      /* DEVICE f32[capacity]                                                */
  const uint32_t* count; /* DEVICE u32: entries written, <= capacity                            */
  uint32_t capacity;     /* = dgs_config.pull_all_capacity                                      */
} dgs_var_packet;

enum {
  DGS_KEEP_LOCAL_MODEL = 1u << 0, /* keep theta_k per worker and add every pulled G to it (Eq. 5) */
  DGS_RESIDUAL_MODE = 1u << 1,    /* worker rule of Algorithm 1 instead of Algorithm 3: v <- v + eta*grad,
                                     sent entries leave v, the rest stay (no momentum, no 1/m rescale) */
  DGS_HOST_IO = 1u << 2,          /* reserve staging buffers for dgs_event_host */
  DGS_NO_SPECULATION = 1u << 3,   /* always take the two-pass selection (histogram pass, then stream pass) */
  DGS_SINGLE_STREAM = 1u << 4,    /* enqueue every step on ONE internal stream: kernels run one after the other in
                                     call order (same results; for debugging and for timing a kernel on its own) */
  DGS_PACKET_BF16 = 1u << 6,      /* packets carry values rounded to bfloat16 (see "16-bit packet values" below)  */
  DGS_PACKET_FP16 = 1u << 7,      /* ... to IEEE binary16, saturating at 65504; not together with DGS_PACKET_BF16  */
  DGS_TEST_STALLED_BARRIER = 1u << 5 /* testing only: the barrier among the CTAs of the finalize kernels waits for one
                                     CTA that does not exist, with a limit of a few thousand polls.  Every wait then
                                     runs out: the kernels return early, packets and state are NOT valid, and
                                     dgs_status reports DGS_ETIMEOUT.  Shows that a wait that cannot end costs a
                                     status word, not the GPU. */
};

typedef struct {
  uint64_t n;                  /* number of parameters, 1 <= n < 2^32                                  */
  uint32_t num_workers;        /* N >= 1                                                               */
  float lr;                    /* eta, finite                                                          */
  float momentum;              /* m, 0 < m <= 1 (1/m is taken once, by IEEE division)                  */
  uint32_t num_segments;       /* S >= 1, S < 65536                                                    */
  const dgs_segment* segments; /* HOST array [S], copied                                               */
  const float* theta0;         /* DEVICE f32[n], initial model (Algorithm 3, first line), copied       */
  void* arena;                 /* DEVICE memory owned by the caller, 256-byte aligned                  */
  uint64_t arena_bytes;        /* >= what dgs_arena_bytes reports for this configuration               */
  void* stream;                /* cudaStream_t on which all work is enqueued (NULL = default stream)   */
  uint32_t flags;              /* DGS_* flags above                                                    */
  uint32_t pull_all_capacity;  /* most entries a dgs_worker_pull_all packet can carry (0: that call is not
                                  used and no packet slots are set aside for it); at most n              */
} dgs_config;

enum { DGS_THETA = 0, DGS_U = 1, DGS_D = 2, DGS_THETA_LOCAL = 3 };

/* Bytes of device memory a context for this configuration carves from the arena
 * (model, N velocities + spares, N differences, packet slots, the log of applied
 * packets, selection scratch).  No GPU work.  arena/arena_bytes/theta0/stream are ignored. */
int dgs_arena_bytes(const dgs_config* cfg, uint64_t* out_bytes);

/* Creates the context: u_k = 0 and D_k = 0 for every worker (Algorithm 3 and
 * Algorithm 2, initialisation), theta = theta0, theta_k = theta0 if kept.
 * Enqueues the clears and copies on cfg->stream.  The arena must stay alive and
 * untouched by others until dgs_free. */
int dgs_init(const dgs_config* cfg, dgs_ctx** out);

/* Worker push (Algorithm 3, velocity update through encode(); Eq. 11a, Eq. 12).
 * grad: DEVICE f32[n], 16-byte aligned, read only, must stay valid until the work of
 * this call has run (dgs_flush, then the stream reaching that point).  On return *out
 * describes the push packet slot (a few slots are used in turn). */
int dgs_worker_push(dgs_ctx* ctx, uint32_t worker, const float* grad, dgs_packet* out);

/* Server apply (Algorithm 2, "M <- M - decode(g)"; Eq. 1-3): theta[i] -= val and
 * D_q[i] -= val for every worker q, the sender included, for each (i, val) of the
 * packet.  pkt may be the library's own push packet or any DEVICE packet with
 * strictly ascending indices < n.  Also advances the server timestamp t.
 * For the library's own packets the subtraction from D_q is deferred: the packet is
 * filed in a log and folded into D_q, in arrival order, before anything reads D_q
 * (that worker's next pull, dgs_state_ptr); every D_q[i] sees the same subtractions
 * in the same order, so the values are the same bit for bit. */
int dgs_server_apply(dgs_ctx* ctx, uint32_t worker, const dgs_packet* pkt);

/* Worker pull with secondary compression (Algorithm 2, per-layer top-k of
 * G = M - v_k; Eq. 6a, 6b): builds the pull packet from D_worker, clears the sent
 * entries there, adds them to theta_worker when DGS_KEEP_LOCAL_MODEL is set
 * (Eq. 5), and records prev(worker) = t. */
int dgs_worker_pull(dgs_ctx* ctx, uint32_t worker, dgs_packet* out);

/* Worker pull WITHOUT secondary compression (Algorithm 2 with the switch off, the paper's
 * normal case; Eq. 3, Eq. 4): the packet lists every entry of D_worker that is not zero (+0 and
 * -0 both count as zero), in ascending index order, and those entries are cleared, so that
 * v_worker = M afterwards; they are added to theta_worker when DGS_KEEP_LOCAL_MODEL is set
 * (Eq. 5); prev(worker) = t.  The number of entries is written to a device word of the packet
 * slot (no host synchronisation); *out is filled at once.  If D_worker holds more nonzero
 * entries than cfg.pull_all_capacity, the first `capacity` of them (lowest indices) are sent
 * and cleared, the others stay in D_worker for a later pull, and the device status word
 * becomes DGS_ELIMIT (see dgs_status).  Needs pull_all_capacity > 0, else DGS_EINVAL.  A few
 * packet slots are used in turn: a packet stays valid until the fourth later call. */
int dgs_worker_pull_all(dgs_ctx* ctx, uint32_t worker, dgs_var_packet* out);

/* One whole event for `worker`: push, apply of that packet, pull.  Either packet
 * pointer may be NULL. */
int dgs_event(dgs_ctx* ctx, uint32_t worker, const float* grad, dgs_packet* push_out, dgs_packet* pull_out);

/* Makes the stream given at dgs_init wait (on the device, not the host) for all work
 * enqueued by earlier calls: what that stream runs afterwards sees their packets and
 * state.  (No counterpart in the paper: it joins the library's own streams -- four for the
 * pushes, one for the apply, six for the pulls -- to the caller's.) */
int dgs_flush(dgs_ctx* ctx);

/* The same event with HOST buffers (needs DGS_HOST_IO): copies grad (HOST f32[n],
 * ideally pinned) to the device, runs the event, copies the pull packet back into
 * out_idx / out_val (HOST, sum(k_pull) entries each, may be NULL to skip) and
 * waits for that work.  This is the end-to-end path: what a worker process
 * without its own device buffers would call. */
int dgs_event_host(dgs_ctx* ctx, uint32_t worker, const float* grad_host, uint32_t* out_idx, float* out_val);

/* Pointer to a state vector, DEVICE f32[n]: which = DGS_THETA (worker ignored),
 * DGS_U, DGS_D or DGS_THETA_LOCAL.  Waits for all work in flight (velocity buffers are
 * exchanged with a spare on the device, so their address is only known then).
 * The pointer is valid until the next push of that worker (DGS_U) or dgs_free. */
int dgs_state_ptr(dgs_ctx* ctx, int which, uint32_t worker, const float** out);

/* Overwrites a state vector from src (DEVICE f32[n]) on the stream: restores a
 * checkpoint, or loads a vector to be selected from with dgs_worker_pull. */
int dgs_state_load(dgs_ctx* ctx, int which, uint32_t worker, const float* src);

/* Waits for all work in flight and returns the sticky device status word in
 * *device_status (0 = clean; negative dgs_error values are stored by kernels that
 * detect an out-of-range index or give up a bounded wait). */
int dgs_status(dgs_ctx* ctx, int* device_status);

/* Waits for all work in flight and reports counters: out[0] selections served by the
 * single-pass (speculative) route, out[1] selections that took the two-pass
 * route from the start or started over because the carried bound admitted fewer
 * than k candidates, out[2] server timestamp t (packets applied), out[3] candidates
 * the finalize steps have examined in total (the k selected ones included). */
int dgs_stats(dgs_ctx* ctx, uint64_t out[4]);

/* Waits for all work in flight and reports how much of the difference vectors the pulls'
 * stream passes had to read: out[0] stage-sized chunks (4096 elements) of whole tiles that
 * the passes covered, out[1] those of them that were actually read.  The library keeps,
 * per 512 elements of every D_q, an upper bound on the magnitudes in it; a chunk whose
 * bounds are all below the selection's lower bound cannot hold a selected entry (Eq. 6a
 * takes the largest magnitudes) and is not read.  The selection stays exact. */
int dgs_pull_read_stats(dgs_ctx* ctx, uint64_t out[2]);

/* prev(worker): the server timestamp at that worker's last pull, -1 before it. */
int dgs_prev(dgs_ctx* ctx, uint32_t worker, int64_t* out);

/* Number of kernels this context has launched so far (host-side count). */
int dgs_launch_count(dgs_ctx* ctx, uint64_t* out);

/* Kernels the library launches, as indices into the arrays of dgs_timing_read. */
enum {
  DGS_KERNEL_STREAM_PUSH = 0,   /* push, single-pass route: velocity update + candidate collection      */
  DGS_KERNEL_FINALIZE_PUSH = 1, /* push, single-pass route: exact k-th key, ordered packet, fix-ups      */
  DGS_KERNEL_TWO_PASS_PUSH = 2, /* push, two-pass route only: histogram of the whole input + bound pick  */
  DGS_KERNEL_SCATTER = 3,       /* apply: theta -= packet, packet filed in the log (or the eager scatter) */
  DGS_KERNEL_STREAM_PULL = 4,
  DGS_KERNEL_FINALIZE_PULL = 5,
  DGS_KERNEL_TWO_PASS_PULL = 6,
  DGS_KERNEL_CATCH_UP = 7,      /* pull: filed packets folded into the worker's difference vector        */
  DGS_NUM_KERNELS = 8
};

/* Measurement aid (no counterpart in the paper).  While on, every kernel launch of
 * this context is bracketed by two CUDA events on the stream it runs on (at most
 * 65536 launches between two reads are recorded). */
int dgs_timing_enable(dgs_ctx* ctx, int on);

/* Waits for all work in flight; ms[i] / count[i] receive the summed device time in
 * milliseconds and the number of recorded launches of kernel i since the last
 * read, and the accumulators restart from zero. */
int dgs_timing_read(dgs_ctx* ctx, double ms[DGS_NUM_KERNELS], uint64_t count[DGS_NUM_KERNELS]);

/* Measurement aid (no counterpart in the paper): the launches recorded since the last read as
 * a timeline instead of sums.  Waits for all work in flight.  For the first min(cap, recorded)
 * launches, in the order they were enqueued: start_ms / stop_ms (HOST f32[cap]) receive the
 * device times of the two events around the launch, in milliseconds after the first recorded
 * launch began; kernel[i] one of DGS_KERNEL_*; stream[i] the index of the library stream it
 * ran on.  *count receives how many entries were written.  The record restarts empty (the sums
 * of dgs_timing_read do not include these launches). */
int dgs_timing_trace(dgs_ctx* ctx, uint32_t cap, float* start_ms, float* stop_ms, int32_t* kernel, int32_t* stream,
                     uint32_t* count);

/* How many hardware queues the library's streams want (*needed: its own streams plus the caller's)
 * and how many the process asked the driver for (*configured: CUDA_DEVICE_MAX_CONNECTIONS as the
 * process environment has it now, 8 if unset or unreadable).  configured < needed means that some of
 * the library's streams share a queue and their kernels do not overlap.  No GPU work; either
 * pointer may be NULL.  (No counterpart in the paper.) */
int dgs_hardware_queues(int* needed, int* configured);

/* The cudaError_t of the last failed runtime call of this context (0 if none). */
int dgs_last_cuda_error(dgs_ctx* ctx);

/* Frees the host-side context.  The arena stays the caller's.  Waits for all work in flight. */
int dgs_free(dgs_ctx* ctx);

/* Largest vector dgs_topk_encode_static accepts (elements). */
#define DGS_STATIC_MAX_N (1u << 20)

/* Top-k selection and coordinate-format encoding of one flat vector, for callers that
 * must not allocate.  (No counterpart in the paper: this is the selection + encode() step
 * of dgs_worker_pull offered on its own, for one layer, without a context.)
 *
 * Who needs it: code that runs where device allocation is off limits -- inside a region
 * whose memory plan is frozen (a pre-sized pool that must not grow, a real-time or
 * serving loop that may not call into the allocator), or a plug-in that is handed
 * buffers but no allocator.  Such a caller cannot give dgs_init an arena either.  Here
 * every byte of scratch (a private copy of x, the candidate list, histograms, the
 * barrier words: about 12.6 MB) lives in one fixed array that is part of the library's
 * device image; each GPU that loads the library holds it until the process exits.
 *
 *   x        DEVICE f32[n], read only
 *   n, k     1 <= k <= n <= DGS_STATIC_MAX_N; a larger n returns DGS_ELIMIT, other bad
 *            arguments DGS_EINVAL, and nothing is enqueued
 *   out_idx  DEVICE u32[k], out_val DEVICE f32[k]: the k entries of largest |x| (ties to
 *            the lowest index), ascending index, exactly as dgs_worker_pull would list them
 *   stream   cudaStream_t; the work is enqueued there and the call returns
 *
 * The function calls no cudaMalloc / cudaFree and no allocating library routine.  The
 * first call on each device looks up the address of the array for that device (the
 * device must be current, as for every call) and sizes its launches; make that first
 * call outside any stream capture.  All calls on a device share the one array: it keeps
 * what the previous call left, the function clears what has to start at zero itself, and
 * two calls whose work overlaps on the GPU (different streams, no ordering) race on it --
 * order them. */
int dgs_topk_encode_static(const float* x, uint32_t n, uint32_t k, uint32_t* out_idx, float* out_val, void* stream);

/* Device-side outcome of the dgs_topk_encode_static calls enqueued on `stream` so far.  (No
 * counterpart in the paper.)  dgs_topk_encode_static only enqueues work, so it cannot report a
 * failure that happens on the device: a bounded wait that gave up (DGS_ETIMEOUT) or an
 * internal rank check that failed leave out_idx / out_val partly unwritten.  This call waits
 * for `stream` (host-side wait), then stores in *device_status the status word of the last
 * call's kernels: 0 = the packet is complete, negative = it is not.  Like the selection itself
 * it allocates nothing (one 4-byte copy from the fixed array). */
int dgs_topk_encode_static_status(void* stream, int* device_status);

/* Static text for a dgs_error value. */
const char* dgs_error_string(int err);

#ifdef __cplusplus
}
#endif
#endif /* DGS_H_ */
