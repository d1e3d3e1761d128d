/* dcasgd.h - C ABI of the DC-ASGD parameter-server update for NVIDIA B200 (sm_100a).
 *
 * The library is the SERVER of "Asynchronous Stochastic Gradient Descent with Delay
 * Compensation" (Zheng et al., arXiv 1609.08326): Algorithm 2, with the update rule of
 * Section 4 (Eq. 10) and the adaptive lambda of Section 6 (the "MeanSquare" equation).  The
 * workers of Algorithm 1 are the callers: a "message" is a function call that carries a device
 * pointer.
 *
 *   state      w[n]              the global model                          (fp32, device)
 *              w_bak[M][stride]  one backup per worker, Algorithm 2        (fp32, device)
 *              ms[n]             MeanSquare, adaptive variant only         (fp32, device)
 *              t                 number of gradients applied so far        (host)
 *
 *   pull(m)    w_bak[m] <- w                                              Algorithm 2, pull branch
 *   push(m,g)  w <- w - eta*( g + lambda_t * g.g.(w - w_bak[m]) ); t <- t+1  Algorithm 2, gradient branch; Eq. 10
 *              constant variant (DC-ASGD-c): lambda_t = lambda
 *              adaptive variant (DC-ASGD-a): ms <- mu*ms + (1-mu)*g.g ;  lambda_t = lambda / sqrt(ms + eps)
 *
 *   momentum   (optional; Section 6 mentions momentum variants in a footnote and prints no formula.
 *              Reading: classical momentum on the delay-compensated gradient u = g + lambda_t*g.g.(w - w_bak[m]):
 *              v <- beta*v + eta*u ;  w <- w - v ;  v starts at 0; beta = 0 is Eq. 10 itself)
 *
 * Arithmetic: IEEE binary32, every operation rounded to nearest on its own (no fused
 * multiply-add), in this order per element:
 *     gg = g*g ; [ms = mu*ms + (1-mu)*gg ; lam = lambda / sqrt(ms + eps)] ;
 *     d = w - w_bak[m] ; c = (lam*gg)*d ; u = g + c ; w = w - eta*u
 *     (momentum: p = eta*u ; v = beta*v + p ; w = w - v)
 * with (1-mu) rounded once on the host.  bfloat16 gradients are widened exactly first.  Results
 * therefore do not depend on which kernel (single push or fused window) applied an event.
 *
 * Conventions
 *   Pointers   "device" pointers must be valid on the CUDA device that is current when
 *              dcasgd_create runs; "host" pointers are ordinary process memory.
 *   Ownership  The library BORROWS every device buffer (the caller allocates, e.g. with
 *              PyTorch, and keeps them alive until dcasgd_destroy).  It owns only the handle.
 *              It never allocates device memory.  Host arrays are read during the call only.
 *   Ordering   Every call enqueues its kernels on cfg.stream and returns without
 *              synchronising.  The serial order of Algorithm 2 is the stream order.
 *   Errors     Every function returns a dcasgd_status.  All arguments and every log record are
 *              validated on the host BEFORE anything is launched: a call that fails with a
 *              status other than DCASGD_ECUDA has changed nothing.  Nothing aborts, throws or
 *              traps.  dcasgd_last_error() gives the text of the calling thread's last failure.
 *   Threads    One server handle is used by one host thread at a time.
 *   Legal      A push with no earlier pull (the backup still holds w_0), repeated pushes on one
 *              pull, repeated pulls: Algorithm 2 has no rule against them, neither has this.
 *   Tuning     Read by dcasgd_create from the environment; none changes a result, only speed.
 *              DCASGD_REPLAY_VECS=1|2      16-byte vectors per thread in the fused kernel
 *              DCASGD_TWO_VEC_SLOTS=k      windows with more than k live snapshots run one vector per thread (default 8)
 *              DCASGD_WINDOW_SLOTS=k       live snapshots a window may keep before it is cut (default 16)
 *              DCASGD_IEEE_LIBRARY_MATH=1  adaptive lambda always through the compiler's sqrt and division
 */
#ifndef DCASGD_H
#define DCASGD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DCASGD_VERSION 0x00010000u

typedef struct dcasgd_server dcasgd_server; /* opaque */

typedef enum {
  DCASGD_OK = 0,
  DCASGD_EINVAL = 1,  /* NULL where a pointer is required, bad enum, non-finite hyper-parameter, overlap */
  DCASGD_EWORKER = 2, /* worker index >= num_workers */
  DCASGD_EALIGN = 3,  /* pointer or stride not aligned as documented */
  DCASGD_ELOG = 4,    /* malformed log record (kind, worker, grad_id, eta) */
  DCASGD_ECUDA = 5,   /* CUDA runtime error; text in dcasgd_last_error() */
  DCASGD_ENOMEM = 6   /* host allocation failed */
} dcasgd_status;

enum { DCASGD_CONST = 0, DCASGD_ADAPTIVE = 1 }; /* DC-ASGD-c / DC-ASGD-a (Section 6) */
enum { DCASGD_F32 = 0, DCASGD_BF16 = 1 };       /* storage type of pushed gradients */
enum { DCASGD_PULL = 0, DCASGD_PUSH = 1 };      /* the two messages of Algorithm 2 */
/* dcasgd_config.flags.  DCASGD_RESUME: w, w_bak and ms already hold a saved server state (a
 * checkpoint the caller copied into them): dcasgd_create leaves them as they are instead of
 * running "Initialize"; restore t with dcasgd_set_step. */
enum { DCASGD_RESUME = 1u };

typedef struct {
  uint64_t n;            /* number of parameters; 0 is allowed (every call is then a no-op) */
  uint32_t num_workers;  /* M, 1..65535 */
  uint32_t variant;      /* DCASGD_CONST | DCASGD_ADAPTIVE */
  uint32_t grad_dtype;   /* DCASGD_F32 | DCASGD_BF16 */
  float eta;             /* default learning rate, used when a push passes eta < 0 */
  float lambda;          /* lambda (constant variant) or lambda_0 (adaptive variant); any finite value */
  float mu;              /* the paper's moving-average constant "m", in [0,1); adaptive only */
  float eps;             /* >= 0; the paper uses 1e-7; adaptive only */
  uint32_t flags;        /* 0, or DCASGD_RESUME */
  float *w;              /* device, n floats, 16-byte aligned; holds w_0 on entry */
  float *w_bak;          /* device, num_workers * w_bak_stride floats (every slab is padded to the stride;
                            the padding may be overwritten), 16-byte aligned */
  uint64_t w_bak_stride; /* floats between slabs: >= n and a multiple of 4 */
  float *ms;             /* device, n floats, 16-byte aligned; NULL if and only if DCASGD_CONST */
  void *stream;          /* cudaStream_t; NULL is the legacy default stream */
  float *v;              /* device, n floats, 16-byte aligned: velocity of the momentum variant; NULL = no momentum */
  float beta;            /* momentum coefficient in [0,1); must be 0 when v is NULL */
  uint32_t reserved;     /* 0 */
} dcasgd_config;

/* One record of the server's message log, 16 bytes. */
typedef struct {
  uint8_t kind;     /* DCASGD_PULL | DCASGD_PUSH */
  uint8_t pad[3];   /* ignored */
  uint32_t worker;  /* m */
  uint32_t grad_id; /* PUSH: which buffer of the gradient pool holds g_m; PULL: ignored */
  float eta;        /* PUSH: learning rate of this update, < 0 = the server's default; PULL: ignored */
} dcasgd_event;

/* Algorithm 2, "Initialize": t = 0, w_bak[m] = w for every m, ms = 0, v = 0 (skipped with
 * DCASGD_RESUME).  cfg (host) is copied.  *out receives the handle.  w, w_bak, ms, v must not overlap. */
int dcasgd_create(const dcasgd_config *cfg, dcasgd_server **out);

/* Algorithm 2, pull branch: w_bak[m] <- w.  If out_w (device, n floats, 16-byte aligned, not
 * overlapping the state) is not NULL it also receives w: the model "sent back to worker m". */
int dcasgd_pull(dcasgd_server *s, uint32_t m, float *out_w);

/* Algorithm 2, gradient branch; Eq. 10 (and the MeanSquare rule when adaptive).
 * g: device, n elements of cfg.grad_dtype, 16-byte aligned, not overlapping the state.
 * eta < 0 selects cfg.eta.  Advances t by one. */
int dcasgd_push(dcasgd_server *s, uint32_t m, const void *g, float eta);

/* The repeat-loop of Algorithm 2 over a recorded message log, in log order.
 *   ev            host, count records
 *   grad_pool     device, num_grads gradient buffers of n elements of cfg.grad_dtype, buffer k
 *                 starting k*grad_stride_bytes after grad_pool (16-byte aligned, stride a
 *                 multiple of 16 and, if num_grads > 1, >= the bytes of one buffer)
 *   window_k      1: one kernel per record (dcasgd_pull / dcasgd_push).
 *                 >= 2: the log is cut into windows of at most window_k records and each window
 *                 is applied by ONE kernel in which every element walks the window's records
 *                 with w (and ms) in registers.  Legal because Eq. 10 and MeanSquare are
 *                 elementwise: the serial dependence of Algorithm 2 runs along t per element
 *                 only.  Same results, bit for bit, as window_k = 1.
 * Validation covers the whole log before the first launch.  count = 0 is a no-op. */
int dcasgd_apply_log(dcasgd_server *s, const dcasgd_event *ev, uint64_t count, const void *grad_pool,
                     uint64_t grad_stride_bytes, uint32_t num_grads, uint32_t window_k);

/* Waits for nothing; forgets the handle.  The caller's buffers stay untouched and must outlive
 * any work still queued on the stream.  NULL is accepted. */
int dcasgd_destroy(dcasgd_server *s);

/* t of Algorithm 2 (number of pushes applied, counting queued ones). */
int dcasgd_get_step(const dcasgd_server *s, uint64_t *t);
int dcasgd_set_step(dcasgd_server *s, uint64_t t);

/* Number of kernels this handle has launched so far. */
int dcasgd_get_launch_count(const dcasgd_server *s, uint64_t *launches);

const char *dcasgd_last_error(void);        /* never NULL; valid until the thread's next failing call */
const char *dcasgd_status_string(int status);
uint32_t dcasgd_version(void);

/* Diagnostic, no counterpart in the paper.  For the adaptive variant the kernels compute
 * lambda_t = lambda_0 / sqrt(s), s = ms + eps, on a branch-free route (packed FMAs, one Newton
 * correction for the root, a once-refined reciprocal and one exact-residual correction of the
 * quotient) when s is in [2^-100, 2^100) and
 * |lambda_0| in [2^-60, 2^60), and with the compiler's guarded IEEE sqrt and division otherwise.
 * (The branch-free route was compared with the IEEE one on every pair of significands, see
 * dcasgd_check_adaptive_lambda_grid below: results are bit-equal for EVERY admissible lambda_0.)
 * This call runs both routes on EVERY binary32 value s in [s_first, s_last] for the given
 * lambda_0 and ADDS the number of inputs on which their bits differ to *mismatches_dev (device,
 * 8 bytes, 8-byte aligned, zeroed by the caller).  Enqueued on `stream`; allocates nothing.
 * The expected count is 0 for every admissible argument. */
int dcasgd_check_adaptive_lambda(float lambda0, float s_first, float s_last, void *stream, uint64_t *mismatches_dev);

/* The same comparison over a grid of numerators and radicands: a takes the a_count binary32 values
 * whose encodings are bits(a_first), bits(a_first) + a_step, ... (all of one sign, every |a| in
 * [2^-60, 2^60)), s every binary32 value in [s_first, s_last].  The branch-free route only
 * multiplies, adds and fuses, and nothing in it leaves the normal range for these arguments, so
 * scaling a by 2 or s by 4 scales every intermediate by a power of two: whether it rounds
 * correctly depends on the significands alone.  a in [1, 2) with a_step = 1 (2^23 values) and s
 * in [1, 4) (2^24 values) therefore covers EVERY admissible pair; that run takes a minute or two
 * on a B200 and finds no mismatch.  The work is cut into launches of a fraction of a second. */
int dcasgd_check_adaptive_lambda_grid(float a_first, uint32_t a_count, uint32_t a_step, float s_first, float s_last,
                                      void *stream, uint64_t *mismatches_dev);

/* Checked build, no counterpart in the paper.  A library compiled with -DDCASGD_DEBUG_CHECKS
 * makes every kernel compare each global-memory address it is about to use with the buffers of
 * the call (the server's w / w_bak / ms / v and the caller's g, out_w or gradient pool, with the
 * extents the host validated).  An access outside all of them, a store into a read-only buffer
 * or a misaligned access is skipped - nothing traps, nothing faults - and a bit is ORed into
 * *status_dev (device, 4 bytes, 4-byte aligned, zeroed by the caller): 1 = bad read,
 * 2 = bad write, 4 = misaligned.  With a server handle the word serves that server from its
 * next launch on; with s = NULL it becomes the default that servers created afterwards (and the
 * lambda self-check) inherit, so that "Initialize" is covered too.  status_dev = NULL stops the
 * recording (violating accesses are still skipped).  The access table sits in constant memory
 * and is replaced in stream order before each launch: use one stream at a time in this build.
 * In the normal build no check exists in the kernels and this call returns DCASGD_EINVAL. */
int dcasgd_debug_checks(dcasgd_server *s, uint32_t *status_dev);

/* ---- window compiler (host only; no CUDA call) -------------------------------------------
 * What dcasgd_apply_log does to a window before launching, exposed so that it can be
 * inspected and tested without a GPU.  A window of the log becomes a list of STEPS.  Step 0 has
 * no push; step j (1..n_pushes) applies push j-1.  After the push of a step, w is a value that
 * the pulls recorded before the next push all copy; the program keeps what is needed of them:
 *   - src[j-1] >= 0 : push j-1 measures its delay against w_bak[src] as it was BEFORE the window
 *                     (read from memory); src < 0 : against in-window snapshot slot -(src+1)
 *   - save_slot[j]  : slot that receives w after step j, or -1
 *   - store_worker[store_begin[j] .. store_begin[j+1]) : workers whose LAST pull of the window
 *                     comes after step j; w is written to their w_bak slab.  Pulls that are
 *                     superseded inside the window without being used cost nothing.
 * The window is shortened (n_records < window_k) when it would need more than
 * max_slots (at most DCASGD_MAX_WINDOW_SLOTS) live snapshots, DCASGD_MAX_WINDOW_PUSHES pushes or
 * DCASGD_MAX_WINDOW_STORES stores; the remaining records start the next window.  (The program
 * travels to the kernel as a launch parameter: a window of up to 128 pushes and 192 stores in
 * a 5.6 KB form, a longer one in a 28 KB form.  Long windows pay off where the vector is short
 * and a launch would otherwise cost as much as the work it carries.) */
#define DCASGD_MAX_WINDOW_PUSHES 640
#define DCASGD_MAX_WINDOW_STORES 960
#define DCASGD_MAX_WINDOW_SLOTS 16

typedef struct {
  uint32_t n_records;       /* log records this window consumed (>= 1) */
  uint32_t n_pushes;        /* P */
  uint32_t n_slots;         /* in-window snapshot slots used */
  uint32_t n_stores;        /* W: backup slabs written */
  uint32_t n_snapshot_reads;/* R: pushes that read a pre-window backup from memory */
  uint32_t n_dead_pulls;    /* pulls that needed no action */
  uint32_t grad_id[DCASGD_MAX_WINDOW_PUSHES];
  float eta[DCASGD_MAX_WINDOW_PUSHES];      /* resolved: never negative */
  int32_t src[DCASGD_MAX_WINDOW_PUSHES];
  int32_t save_slot[DCASGD_MAX_WINDOW_PUSHES + 1];
  uint32_t store_begin[DCASGD_MAX_WINDOW_PUSHES + 2];
  uint32_t store_worker[DCASGD_MAX_WINDOW_STORES];
} dcasgd_window_program;

/* Compiles the window that starts at ev[0] (host, count records available, at most window_k
 * taken), using at most max_slots in-window snapshot slots (0 = DCASGD_MAX_WINDOW_SLOTS).
 * Records must be valid (kind, worker < num_workers); DCASGD_ELOG otherwise. */
int dcasgd_compile_window(const dcasgd_event *ev, uint64_t count, uint32_t num_workers, uint32_t window_k,
                          float default_eta, uint32_t max_slots, dcasgd_window_program *out);

/* The slot limit dcasgd_apply_log passes to the compiler for this server: with it,
 * dcasgd_compile_window cuts a log exactly as dcasgd_apply_log does. */
int dcasgd_get_window_slot_cap(const dcasgd_server *s, uint32_t *max_slots);

#ifdef __cplusplus
}
#endif
#endif /* DCASGD_H */
