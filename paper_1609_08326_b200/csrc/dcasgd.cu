// Host side of the C ABI declared in dcasgd.h: argument validation, the serial message loop of
// Algorithm 2, and the launches.  Every check runs before the first launch of a call.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "dcasgd.h"
#include "kernels.cuh"
#include "window_compiler.h"

using namespace dcasgd;

struct dcasgd_server {
    dcasgd_config cfg;
    Hyper h;
    cudaStream_t stream;
    int device;
    int sms;             // multiprocessors of the device
    int replay_vecs;     // 16-byte vectors per thread in the fused replay kernel (1 or 2) for windows with few slots
    uint32_t two_vec_slots;  // a window that needs more slots than this runs one vector per thread
    uint32_t slot_cap;   // in-window snapshot slots a window may use
    uint64_t t;          // pushes applied (Algorithm 2's t)
    uint64_t launches;   // kernels launched through this handle
    uint32_t* debug_status;  // checked build: device word that collects access violations, or NULL
};

namespace {

struct Range { const char* lo; const char* hi; const char* name; };

inline Range range_of(const void* p, uint64_t bytes, const char* name) {
    return Range{static_cast<const char*>(p), static_cast<const char*>(p) + bytes, name};
}
inline bool overlap(const Range& a, const Range& b) {
    return a.lo < b.hi && b.lo < a.hi && a.lo != a.hi && b.lo != b.hi;
}
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline uint64_t grad_elem_bytes(const dcasgd_config& c) { return c.grad_dtype == DCASGD_BF16 ? 2 : 4; }

int fail(int status, const char* fmt, ...) __attribute__((format(printf, 2, 3)));
int fail(int status, const char* fmt, ...) {
    char buf[400];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    set_error("%s", buf);
    return status;
}

int cuda_fail(const char* what, cudaError_t e) {
    return fail(DCASGD_ECUDA, "%s: %s (%s)", what, cudaGetErrorName(e), cudaGetErrorString(e));
}

// The state arrays of a server as byte ranges, for overlap checks against caller buffers.
int state_ranges(const dcasgd_config& c, Range out[4]) {
    int k = 0;
    out[k++] = range_of(c.w, c.n * 4, "w");
    const uint64_t bak = c.n == 0 ? 0 : (uint64_t)c.num_workers * c.w_bak_stride * 4;   // every slab is stride floats long
    out[k++] = range_of(c.w_bak, bak, "w_bak");
    if (c.ms) out[k++] = range_of(c.ms, c.n * 4, "ms");
    if (c.v) out[k++] = range_of(c.v, c.n * 4, "v");
    return k;
}

int check_foreign(const dcasgd_config& c, const void* p, uint64_t bytes, const char* name) {
    Range st[4];
    const int k = state_ranges(c, st);
    const Range r = range_of(p, bytes, name);
    for (int i = 0; i < k; ++i)
        if (overlap(r, st[i])) return fail(DCASGD_EINVAL, "%s overlaps the server's %s", name, st[i].name);
    return DCASGD_OK;
}

// cuMemGetAddressRange of the driver, looked up through the runtime (the library does not link
// against the driver); NULL when the lookup fails, and the extent check is then skipped.
typedef int (*mem_range_fn)(unsigned long long* base, size_t* size, unsigned long long ptr);
mem_range_fn mem_range() {
    static const mem_range_fn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuMemGetAddressRange", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            f = nullptr;
        }
        return reinterpret_cast<mem_range_fn>(f);
    }();
    return fn;
}

// One address must be device (or managed) memory of device `dev`.
int check_device_address(const char* fn, const char* name, const void* p, int dev) {
    cudaPointerAttributes at;
    const cudaError_t e = cudaPointerGetAttributes(&at, p);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return fail(DCASGD_EINVAL, "%s: %s is not a usable device pointer (%s)", fn, name, cudaGetErrorName(e)); }
    if (at.type != cudaMemoryTypeDevice && at.type != cudaMemoryTypeManaged)
        return fail(DCASGD_EINVAL, "%s: %s is not device memory", fn, name);
    if (at.type == cudaMemoryTypeDevice && at.device != dev)
        return fail(DCASGD_EINVAL, "%s: %s lives on device %d, current device is %d", fn, name, at.device, dev);
    return DCASGD_OK;
}

// A caller buffer [p, p+bytes) must be device memory of device `dev` from its first to its last
// byte: a host pointer, another device's memory or a buffer shorter than stated is refused here,
// on the host, instead of faulting in a kernel.  The extent is checked against the allocation
// that holds p; a buffer that spans several mappings (a virtual-memory pool) is accepted when
// its last byte is device memory of the same device too.
int check_device_buffer(const char* fn, const char* name, const void* p, uint64_t bytes, int dev) {
    if (bytes == 0) return DCASGD_OK;
    int rc = check_device_address(fn, name, p, dev);
    if (rc) return rc;
    const char* last = static_cast<const char*>(p) + (bytes - 1);
    if (mem_range_fn range = mem_range()) {
        unsigned long long base = 0;
        size_t size = 0;
        if (range(&base, &size, (unsigned long long)reinterpret_cast<uintptr_t>(p)) == 0 &&
            reinterpret_cast<uintptr_t>(last) < base + size)
            return DCASGD_OK;
    }
    if (check_device_address(fn, name, last, dev))
        return fail(DCASGD_EINVAL, "%s: %s is shorter than the %llu bytes this call needs", fn, name, (unsigned long long)bytes);
    return DCASGD_OK;
}

inline unsigned blocks_for(uint64_t n, int vecs_per_thread) {
    const uint64_t nvec = (n + 3) / 4;
    const uint64_t per_block = (uint64_t)kThreads * vecs_per_thread;
    return (unsigned)((nvec + per_block - 1) / per_block);
}

#ifdef DCASGD_DEBUG_CHECKS
uint32_t* g_default_debug_status = nullptr;      // inherited by servers created afterwards

// Checked build: before a launch, tell the kernels which address ranges they may touch - the
// server's state arrays (writable) and the caller buffer of this call.  The table lives in
// constant memory and is replaced in stream order, so launches of one stream see their own.
int debug_arm(cudaStream_t stream, const dcasgd_config* c, uint32_t* status, const void* extra, uint64_t extra_bytes,
              bool extra_writable) {
    DebugTable t;
    std::memset(&t, 0, sizeof t);
    auto add = [&t](const void* p, uint64_t bytes, bool writable) {
        if (!p || !bytes) return;
        t.lo[t.n_ranges] = static_cast<const char*>(p);
        t.hi[t.n_ranges] = static_cast<const char*>(p) + bytes;
        if (writable) t.writable |= 1u << t.n_ranges;
        t.n_ranges += 1;
    };
    if (c) {
        Range st[4];
        const int k = state_ranges(*c, st);
        for (int i = 0; i < k; ++i) add(st[i].lo, (uint64_t)(st[i].hi - st[i].lo), true);
    }
    add(extra, extra_bytes, extra_writable);
    // Self-test of the checker: DCASGD_CHECKED_SHRINK=<bytes> makes the TABLE (not the buffers)
    // that much shorter at the end of every range, so the kernels' legitimate last accesses are
    // reported and skipped.  No invalid address is ever touched.
    if (const char* v = std::getenv("DCASGD_CHECKED_SHRINK")) {
        const long k = std::atol(v);
        for (uint32_t i = 0; i < t.n_ranges; ++i)
            if (k > 0 && t.hi[i] - t.lo[i] > k) t.hi[i] -= k;
    }
    t.status = status;
    const cudaError_t e = cudaMemcpyToSymbolAsync(c_dbg, &t, sizeof t, 0, cudaMemcpyHostToDevice, stream);
    return e == cudaSuccess ? DCASGD_OK : cuda_fail("checked build: arming the access table", e);
}
#define DCASGD_DEBUG_ARM(s, extra, bytes, writable)                                                         \
    do { const int rc_ = debug_arm((s)->stream, &(s)->cfg, (s)->debug_status, extra, bytes, writable); if (rc_) return rc_; } while (0)
#else
#define DCASGD_DEBUG_ARM(s, extra, bytes, writable) do { } while (0)
#endif

int after_launch(dcasgd_server* s, const char* what) {
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(what, e);
    s->launches += 1;
    return DCASGD_OK;
}

int launch_pull(dcasgd_server* s, uint32_t m, float* out_w) {
    const dcasgd_config& c = s->cfg;
    if (c.n == 0) return DCASGD_OK;
    DCASGD_DEBUG_ARM(s, out_w, c.n * 4, true);
    k_pull<<<blocks_for(c.n, kPullUnroll), kThreads, 0, s->stream>>>(
        c.w, c.w_bak + (uint64_t)m * c.w_bak_stride, out_w, c.n);
    return after_launch(s, "pull kernel");
}

int launch_push(dcasgd_server* s, uint32_t m, const void* g, float eta) {
    const dcasgd_config& c = s->cfg;
    if (c.n == 0) { s->t += 1; return DCASGD_OK; }
    PushArgs a;
    a.w = c.w;
    a.wb_m = c.w_bak + (uint64_t)m * c.w_bak_stride;
    a.ms = c.ms;
    a.g = g;
    a.vel = c.v;
    a.n = c.n;
    a.eta = eta < 0.0f ? c.eta : eta;
    a.h = s->h;
    const unsigned grid = blocks_for(c.n, kPushUnroll);
    const bool ad = c.variant == DCASGD_ADAPTIVE, bf = c.grad_dtype == DCASGD_BF16, mom = c.v != nullptr;
    DCASGD_DEBUG_ARM(s, g, c.n * grad_elem_bytes(c), false);
#define DCASGD_LAUNCH_PUSH(AD, BF)                                                           \
    do {                                                                                     \
        if (mom) k_push<AD, BF, true><<<grid, kThreads, 0, s->stream>>>(a);                  \
        else     k_push<AD, BF, false><<<grid, kThreads, 0, s->stream>>>(a);                 \
    } while (0)
    if (ad && bf)       DCASGD_LAUNCH_PUSH(true, true);
    else if (ad)        DCASGD_LAUNCH_PUSH(true, false);
    else if (bf)        DCASGD_LAUNCH_PUSH(false, true);
    else                DCASGD_LAUNCH_PUSH(false, false);
#undef DCASGD_LAUNCH_PUSH
    const int rc = after_launch(s, "push kernel");
    if (rc == DCASGD_OK) s->t += 1;              // t counts the pushes that were actually enqueued
    return rc;
}

// Fills the device form of a window program: everything a thread would otherwise compute per
// push is resolved here (byte offsets in the pool and in w_bak, shared-memory offsets of the
// snapshot a push reads and of the slot that keeps w after it).
template <class PROG>
void fill_program(PROG& p, const dcasgd_window_program& wp, const dcasgd_config& c, uint64_t grad_stride_bytes, int V) {
    const int S = replay_stages(V);
    p.n_pushes = wp.n_pushes;
    p.pad = 0;
    p.save_off0 = wp.save_slot[0] >= 0 ? replay_slot_off(V, (uint32_t)wp.save_slot[0]) : kNoSave;
    p.store_end0 = wp.store_begin[1];
    for (uint32_t j = 0; j < wp.n_pushes; ++j) {
        FetchStep& f = p.fetch[j];
        ApplyStep& ap = p.apply[j];
        f.g_off = (uint64_t)wp.grad_id[j] * grad_stride_bytes;
        ap.eta = wp.eta[j];
        if (wp.src[j] >= 0) {                    // staged from memory into this push's stage of the snapshot ring
            f.s_off = (uint64_t)wp.src[j] * c.w_bak_stride * 4;
            ap.snap_off = replay_snap_ring_off(V, j % (uint32_t)S);
        } else {                                 // an in-window slot
            f.s_off = kNoMemorySnapshot;
            ap.snap_off = replay_slot_off(V, (uint32_t)(-(wp.src[j] + 1)));
        }
        ap.save_off = wp.save_slot[j + 1] >= 0 ? replay_slot_off(V, (uint32_t)wp.save_slot[j + 1]) : kNoSave;
        ap.store_end = wp.store_begin[j + 2];
    }
    for (uint32_t k = 0; k < wp.n_stores; ++k) p.store_off[k] = (uint64_t)wp.store_worker[k] * c.w_bak_stride * 4;
}

template <class PROG>
void launch_replay(const dcasgd_server* s, const ReplayArgs& a, const PROG& p, int V, unsigned grid, size_t smem) {
    const dcasgd_config& c = s->cfg;
    const bool ad = c.variant == DCASGD_ADAPTIVE, bf = c.grad_dtype == DCASGD_BF16, mom = c.v != nullptr;
#define DCASGD_LAUNCH_REPLAY(AD, BF)                                                               \
    do {                                                                                           \
        if (mom) {                                                                                 \
            if (V == 2) k_replay<AD, BF, true, 2, PROG><<<grid, kThreads, smem, s->stream>>>(a, p);  \
            else        k_replay<AD, BF, true, 1, PROG><<<grid, kThreads, smem, s->stream>>>(a, p);  \
        } else {                                                                                   \
            if (V == 2) k_replay<AD, BF, false, 2, PROG><<<grid, kThreads, smem, s->stream>>>(a, p); \
            else        k_replay<AD, BF, false, 1, PROG><<<grid, kThreads, smem, s->stream>>>(a, p); \
        }                                                                                          \
    } while (0)
    if (ad && bf)       DCASGD_LAUNCH_REPLAY(true, true);
    else if (ad)        DCASGD_LAUNCH_REPLAY(true, false);
    else if (bf)        DCASGD_LAUNCH_REPLAY(false, true);
    else                DCASGD_LAUNCH_REPLAY(false, false);
#undef DCASGD_LAUNCH_REPLAY
}

int launch_window(dcasgd_server* s, const dcasgd_window_program& wp, const void* grad_pool,
                  uint64_t grad_stride_bytes, uint64_t pool_bytes) {
    const dcasgd_config& c = s->cfg;
    if (c.n == 0) { s->t += wp.n_pushes; return DCASGD_OK; }
    if (wp.n_pushes == 0 && wp.n_stores == 0) return DCASGD_OK;   // nothing survives this window
    // many live snapshots: one vector per thread keeps two CTAs per SM resident (a slot costs half)
    const int V = wp.n_slots > s->two_vec_slots ? 1 : s->replay_vecs;
    ReplayArgs a;
    a.w = c.w;
    a.w_bak = c.w_bak;
    a.ms = c.ms;
    a.vel = c.v;
    a.grad_pool = static_cast<const char*>(grad_pool);
    a.n = c.n;
    a.h = s->h;
    const unsigned grid = blocks_for(c.n, V);
    const size_t smem = replay_smem_bytes(wp.n_slots, V);
    DCASGD_DEBUG_ARM(s, grad_pool, pool_bytes, false);
    (void)pool_bytes;
    if (wp.n_pushes <= (uint32_t)DevProgram::kPushes && wp.n_stores <= (uint32_t)DevProgram::kStores) {
        static thread_local DevProgram p;        // kept off the stack
        fill_program(p, wp, c, grad_stride_bytes, V);
        launch_replay(s, a, p, V, grid, smem);
    } else {
        static thread_local DevProgramLong p;
        fill_program(p, wp, c, grad_stride_bytes, V);
        launch_replay(s, a, p, V, grid, smem);
    }
    const int rc = after_launch(s, "window replay kernel");
    if (rc == DCASGD_OK) s->t += wp.n_pushes;
    return rc;
}

template <bool AD, bool BF, bool MOM, class PROG>
cudaError_t allow_slots_prog() {
    cudaError_t e = cudaFuncSetAttribute(k_replay<AD, BF, MOM, 1, PROG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)replay_smem_bytes(DCASGD_MAX_WINDOW_SLOTS, 1));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(k_replay<AD, BF, MOM, 2, PROG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)replay_smem_bytes(DCASGD_MAX_WINDOW_SLOTS, 2));
}
template <bool AD, bool BF, bool MOM>
cudaError_t allow_slots_one() {
    const cudaError_t e = allow_slots_prog<AD, BF, MOM, DevProgram>();
    return e != cudaSuccess ? e : allow_slots_prog<AD, BF, MOM, DevProgramLong>();
}
template <bool AD, bool BF>
cudaError_t allow_slots() {
    const cudaError_t e = allow_slots_one<AD, BF, false>();
    return e != cudaSuccess ? e : allow_slots_one<AD, BF, true>();
}

int check_server(const dcasgd_server* s, const char* fn) {
    if (!s) return fail(DCASGD_EINVAL, "%s: server is NULL", fn);
    int dev = -1;
    const cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(fn, e);
    if (dev != s->device) return fail(DCASGD_EINVAL, "%s: current device %d is not the server's device %d", fn, dev, s->device);
    return DCASGD_OK;
}

}  // namespace

extern "C" {

const char* dcasgd_last_error(void) { return get_error(); }

const char* dcasgd_status_string(int status) {
    switch (status) {
        case DCASGD_OK: return "DCASGD_OK";
        case DCASGD_EINVAL: return "DCASGD_EINVAL";
        case DCASGD_EWORKER: return "DCASGD_EWORKER";
        case DCASGD_EALIGN: return "DCASGD_EALIGN";
        case DCASGD_ELOG: return "DCASGD_ELOG";
        case DCASGD_ECUDA: return "DCASGD_ECUDA";
        case DCASGD_ENOMEM: return "DCASGD_ENOMEM";
        default: return "DCASGD_<unknown>";
    }
}

uint32_t dcasgd_version(void) { return DCASGD_VERSION; }

int dcasgd_create(const dcasgd_config* cfg, dcasgd_server** out) {
    if (!cfg || !out) return fail(DCASGD_EINVAL, "dcasgd_create: NULL argument");
    *out = nullptr;
    const dcasgd_config& c = *cfg;
    if (c.num_workers == 0 || c.num_workers > 65535u)
        return fail(DCASGD_EINVAL, "dcasgd_create: num_workers must be 1..65535 (got %u)", c.num_workers);
    if (c.variant > DCASGD_ADAPTIVE) return fail(DCASGD_EINVAL, "dcasgd_create: unknown variant %u", c.variant);
    if (c.grad_dtype > DCASGD_BF16) return fail(DCASGD_EINVAL, "dcasgd_create: unknown grad_dtype %u", c.grad_dtype);
    if (c.flags & ~(uint32_t)DCASGD_RESUME) return fail(DCASGD_EINVAL, "dcasgd_create: unknown flags 0x%x", c.flags);
    if (!std::isfinite(c.eta) || c.eta < 0.0f) return fail(DCASGD_EINVAL, "dcasgd_create: eta must be finite and >= 0");
    if (!std::isfinite(c.lambda)) return fail(DCASGD_EINVAL, "dcasgd_create: lambda must be finite");
    const bool adaptive = c.variant == DCASGD_ADAPTIVE;
    if (adaptive) {
        if (!(c.mu >= 0.0f && c.mu < 1.0f)) return fail(DCASGD_EINVAL, "dcasgd_create: mu must be in [0,1)");
        if (!(std::isfinite(c.eps) && c.eps >= 0.0f)) return fail(DCASGD_EINVAL, "dcasgd_create: eps must be finite and >= 0");
        if (!c.ms && c.n) return fail(DCASGD_EINVAL, "dcasgd_create: the adaptive variant needs ms");
    } else if (c.ms) {
        return fail(DCASGD_EINVAL, "dcasgd_create: ms must be NULL for the constant variant");
    }
    if (c.reserved != 0) return fail(DCASGD_EINVAL, "dcasgd_create: reserved must be 0");
    if (c.v) {
        if (!(c.beta >= 0.0f && c.beta < 1.0f)) return fail(DCASGD_EINVAL, "dcasgd_create: beta must be in [0,1)");
    } else if (c.beta != 0.0f) {
        return fail(DCASGD_EINVAL, "dcasgd_create: beta must be 0 without a velocity vector v");
    }
    if (c.n) {
        if (!c.w || !c.w_bak) return fail(DCASGD_EINVAL, "dcasgd_create: w and w_bak are required");
        if (c.w_bak_stride < c.n) return fail(DCASGD_EINVAL, "dcasgd_create: w_bak_stride < n");
        if (c.w_bak_stride % 4) return fail(DCASGD_EALIGN, "dcasgd_create: w_bak_stride must be a multiple of 4 floats");
        if (!aligned16(c.w) || !aligned16(c.w_bak) || (c.ms && !aligned16(c.ms)) || (c.v && !aligned16(c.v)))
            return fail(DCASGD_EALIGN, "dcasgd_create: w, w_bak, ms and v must be 16-byte aligned");
        if (c.n > (uint64_t)1 << 40) return fail(DCASGD_EINVAL, "dcasgd_create: n too large");
        Range st[4];
        const int k = state_ranges(c, st);
        for (int i = 0; i < k; ++i)
            for (int j = i + 1; j < k; ++j)
                if (overlap(st[i], st[j]))
                    return fail(DCASGD_EINVAL, "dcasgd_create: %s overlaps %s", st[i].name, st[j].name);
    }

    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail("dcasgd_create: cudaGetDevice", e);
    if (c.n) {
        Range st[4];
        const int k = state_ranges(c, st);
        for (int i = 0; i < k; ++i) {
            const int rc = check_device_buffer("dcasgd_create", st[i].name, st[i].lo, (uint64_t)(st[i].hi - st[i].lo), dev);
            if (rc) return rc;
        }
    }
    if ((e = allow_slots<false, false>()) != cudaSuccess || (e = allow_slots<false, true>()) != cudaSuccess ||
        (e = allow_slots<true, false>()) != cudaSuccess || (e = allow_slots<true, true>()) != cudaSuccess)
        return cuda_fail("dcasgd_create: cudaFuncSetAttribute", e);

    dcasgd_server* s = new (std::nothrow) dcasgd_server;
    if (!s) return fail(DCASGD_ENOMEM, "dcasgd_create: out of host memory");
    s->cfg = c;
    // Route of the adaptive lambda (see kernels.cuh).  The branch-free route is exact for
    // |lambda_0| in [2^-60, 2^60) and s in [2^-100, 2^100).  The lower bound on s needs no test when
    // eps >= 2^-100 and MeanSquare starts at 0 here (it is a sum of non-negative terms from then
    // on); a resumed state comes from the caller, so its MeanSquare is not taken on trust.
    const float al = std::fabs(c.lambda);
    uint32_t route = kLambdaLibrary;
    if (al >= 0x1p-60f && al < 0x1p60f)
        route = (adaptive && c.eps >= 0x1p-100f && !(c.flags & DCASGD_RESUME)) ? kLambdaFloored : kLambdaChecked;
    if (const char* v = std::getenv("DCASGD_IEEE_LIBRARY_MATH")) { if (std::atoi(v) == 1) route = kLambdaLibrary; }
    s->h = make_hyper(c.lambda, adaptive ? c.mu : 0.0f, adaptive ? c.eps : 0.0f, c.v ? c.beta : 0.0f, route);
    s->stream = static_cast<cudaStream_t>(c.stream);
    s->device = dev;
    s->t = 0;
    s->launches = 0;
    s->debug_status = nullptr;
#ifdef DCASGD_DEBUG_CHECKS
    s->debug_status = g_default_debug_status;
#endif
    // Two vectors per thread (3 CTAs/SM, 3-stage ring) measured 4-6 % faster on B200 than one vector
    // per thread (4 CTAs/SM, 5-stage ring) once the vector is long enough to fill the GPU with
    // the larger CTAs (the per-push control work is shared by 8 elements); short vectors keep one
    // vector per thread for the parallelism.  DCASGD_REPLAY_VECS=1|2 overrides the choice.
    int sms = 148;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { (void)cudaGetLastError(); sms = 148; }
    s->sms = sms;
    s->replay_vecs = blocks_for(c.n, 2) >= 2u * (unsigned)sms ? 2 : 1;
    if (const char* v = std::getenv("DCASGD_REPLAY_VECS")) { const int k = std::atoi(v); if (k == 1 || k == 2) s->replay_vecs = k; }
    // A slot costs 4 KB (8 KB with two vectors per thread) of shared memory per CTA on top of the
    // staging ring.  Windows that keep up to 8 snapshots run two vectors per thread (2-3 CTAs per
    // SM); longer windows over many workers need up to 16 and run one vector per thread (2 CTAs
    // per SM), which measured faster than cutting them at 8 slots.
    s->two_vec_slots = 8;
    if (const char* v = std::getenv("DCASGD_TWO_VEC_SLOTS")) { const int k = std::atoi(v); if (k >= 0 && k <= DCASGD_MAX_WINDOW_SLOTS) s->two_vec_slots = (uint32_t)k; }
    s->slot_cap = DCASGD_MAX_WINDOW_SLOTS;
    if (const char* v = std::getenv("DCASGD_WINDOW_SLOTS")) { const int k = std::atoi(v); if (k >= 1 && k <= DCASGD_MAX_WINDOW_SLOTS) s->slot_cap = (uint32_t)k; }
    if (c.n && !(c.flags & DCASGD_RESUME)) {
        // Algorithm 2, Initialize: every backup starts as w_0; MeanSquare(0) = 0
#ifdef DCASGD_DEBUG_CHECKS
        if (const int rc = debug_arm(s->stream, &s->cfg, s->debug_status, nullptr, 0, false)) { delete s; return rc; }
#endif
        k_init<<<blocks_for(c.n, 1), kThreads, 0, s->stream>>>(c.w, c.w_bak, c.w_bak_stride, c.num_workers, c.ms, c.v, c.n);
        const int rc = after_launch(s, "init kernel");
        if (rc != DCASGD_OK) { delete s; return rc; }
    }
    *out = s;
    return DCASGD_OK;
}

int dcasgd_pull(dcasgd_server* s, uint32_t m, float* out_w) {
    int rc = check_server(s, "dcasgd_pull");
    if (rc) return rc;
    if (m >= s->cfg.num_workers) return fail(DCASGD_EWORKER, "dcasgd_pull: worker %u >= %u", m, s->cfg.num_workers);
    if (out_w && s->cfg.n) {
        if (!aligned16(out_w)) return fail(DCASGD_EALIGN, "dcasgd_pull: out_w must be 16-byte aligned");
        if ((rc = check_foreign(s->cfg, out_w, s->cfg.n * 4, "out_w"))) return rc;
        if ((rc = check_device_buffer("dcasgd_pull", "out_w", out_w, s->cfg.n * 4, s->device))) return rc;
    }
    return launch_pull(s, m, out_w);
}

int dcasgd_push(dcasgd_server* s, uint32_t m, const void* g, float eta) {
    int rc = check_server(s, "dcasgd_push");
    if (rc) return rc;
    if (m >= s->cfg.num_workers) return fail(DCASGD_EWORKER, "dcasgd_push: worker %u >= %u", m, s->cfg.num_workers);
    if (!std::isfinite(eta)) return fail(DCASGD_EINVAL, "dcasgd_push: eta is not finite");
    if (s->cfg.n) {
        if (!g) return fail(DCASGD_EINVAL, "dcasgd_push: g is NULL");
        if (!aligned16(g)) return fail(DCASGD_EALIGN, "dcasgd_push: g must be 16-byte aligned");
        if ((rc = check_foreign(s->cfg, g, s->cfg.n * grad_elem_bytes(s->cfg), "g"))) return rc;
        if ((rc = check_device_buffer("dcasgd_push", "g", g, s->cfg.n * grad_elem_bytes(s->cfg), s->device))) return rc;
    }
    return launch_push(s, m, g, eta);
}

int dcasgd_apply_log(dcasgd_server* s, const dcasgd_event* ev, uint64_t count, const void* grad_pool,
                     uint64_t grad_stride_bytes, uint32_t num_grads, uint32_t window_k) {
    int rc = check_server(s, "dcasgd_apply_log");
    if (rc) return rc;
    const dcasgd_config& c = s->cfg;
    if (window_k == 0) return fail(DCASGD_EINVAL, "dcasgd_apply_log: window_k must be >= 1");
    if (count == 0) return DCASGD_OK;
    if (!ev) return fail(DCASGD_EINVAL, "dcasgd_apply_log: ev is NULL");
    // the whole log is checked before anything is launched
    bool any_push = false;
    for (uint64_t r = 0; r < count; ++r) {
        if (ev[r].kind > DCASGD_PUSH) return fail(DCASGD_ELOG, "log record %llu: unknown kind %u", (unsigned long long)r, ev[r].kind);
        if (ev[r].worker >= c.num_workers) return fail(DCASGD_ELOG, "log record %llu: worker %u >= %u", (unsigned long long)r, ev[r].worker, c.num_workers);
        if (ev[r].kind == DCASGD_PUSH) {
            any_push = true;
            if (ev[r].grad_id >= num_grads) return fail(DCASGD_ELOG, "log record %llu: grad_id %u >= %u", (unsigned long long)r, ev[r].grad_id, num_grads);
            if (!std::isfinite(ev[r].eta)) return fail(DCASGD_ELOG, "log record %llu: eta is not finite", (unsigned long long)r);
        }
    }
    const uint64_t gbytes = c.n * grad_elem_bytes(c);
    uint64_t pool_extent = 0;
    if (any_push && c.n) {
        if (!grad_pool) return fail(DCASGD_EINVAL, "dcasgd_apply_log: grad_pool is NULL");
        if (!aligned16(grad_pool) || grad_stride_bytes % 16) return fail(DCASGD_EALIGN, "dcasgd_apply_log: grad_pool and grad_stride_bytes must be multiples of 16 bytes");
        if (num_grads > 1 && grad_stride_bytes < gbytes) return fail(DCASGD_EINVAL, "dcasgd_apply_log: grad_stride_bytes smaller than one gradient");
        const uint64_t pool_bytes = (uint64_t)(num_grads - 1) * grad_stride_bytes + gbytes;
        if ((rc = check_foreign(c, grad_pool, pool_bytes, "grad_pool"))) return rc;
        if ((rc = check_device_buffer("dcasgd_apply_log", "grad_pool", grad_pool, pool_bytes, s->device))) return rc;
        pool_extent = pool_bytes;
    }

    if (window_k == 1) {
        for (uint64_t r = 0; r < count; ++r) {
            if (ev[r].kind == DCASGD_PULL) rc = launch_pull(s, ev[r].worker, nullptr);
            else rc = launch_push(s, ev[r].worker, static_cast<const char*>(grad_pool) + (uint64_t)ev[r].grad_id * grad_stride_bytes, ev[r].eta);
            if (rc) return rc;
        }
        return DCASGD_OK;
    }

    try {
        WindowCompiler wc(c.num_workers);
        dcasgd_window_program wp;
        uint64_t r = 0;
        while (r < count) {
            if ((rc = wc.compile(ev + r, count - r, window_k, c.eta, s->slot_cap, &wp))) return rc;
            if ((rc = launch_window(s, wp, grad_pool, grad_stride_bytes, pool_extent))) return rc;
            r += wp.n_records;
        }
    } catch (const std::bad_alloc&) {
        return fail(DCASGD_ENOMEM, "dcasgd_apply_log: out of host memory");
    }
    return DCASGD_OK;
}

int dcasgd_destroy(dcasgd_server* s) {
    delete s;
    return DCASGD_OK;
}

int dcasgd_get_step(const dcasgd_server* s, uint64_t* t) {
    if (!s || !t) return fail(DCASGD_EINVAL, "dcasgd_get_step: NULL argument");
    *t = s->t;
    return DCASGD_OK;
}

int dcasgd_set_step(dcasgd_server* s, uint64_t t) {
    if (!s) return fail(DCASGD_EINVAL, "dcasgd_set_step: server is NULL");
    s->t = t;
    return DCASGD_OK;
}

int dcasgd_check_adaptive_lambda(float lambda0, float s_first, float s_last, void* stream, uint64_t* mismatches_dev) {
    if (!mismatches_dev) return fail(DCASGD_EINVAL, "dcasgd_check_adaptive_lambda: mismatches_dev is NULL");
    const float al = std::fabs(lambda0);
    if (!(al >= 0x1p-60f && al < 0x1p60f)) return fail(DCASGD_EINVAL, "dcasgd_check_adaptive_lambda: |lambda0| must be in [2^-60, 2^60)");
    if (!(s_first >= 0x1p-100f && s_last < 0x1p100f && s_first <= s_last))
        return fail(DCASGD_EINVAL, "dcasgd_check_adaptive_lambda: need 2^-100 <= s_first <= s_last < 2^100");
    if (reinterpret_cast<uintptr_t>(mismatches_dev) & 7u)
        return fail(DCASGD_EALIGN, "dcasgd_check_adaptive_lambda: mismatches_dev must be 8-byte aligned");
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail("dcasgd_check_adaptive_lambda: cudaGetDevice", e);
    if (const int rc = check_device_buffer("dcasgd_check_adaptive_lambda", "mismatches_dev", mismatches_dev, 8, dev)) return rc;
    int sms = 148;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { (void)cudaGetLastError(); sms = 148; }
    uint32_t b0, b1;
    std::memcpy(&b0, &s_first, 4);
    std::memcpy(&b1, &s_last, 4);
#ifdef DCASGD_DEBUG_CHECKS
    if (const int rc = debug_arm(static_cast<cudaStream_t>(stream), nullptr, g_default_debug_status, mismatches_dev, 8, true)) return rc;
#endif
    k_check_lambda<<<(unsigned)sms * 8, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        make_hyper(lambda0, 0.0f, 0.0f, 0.0f, kLambdaChecked), b0, (uint64_t)b1 - b0 + 1, reinterpret_cast<unsigned long long*>(mismatches_dev));
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail("lambda self-check kernel", e);
    return DCASGD_OK;
}

int dcasgd_check_adaptive_lambda_grid(float a_first, uint32_t a_count, uint32_t a_step, float s_first, float s_last,
                                      void* stream, uint64_t* mismatches_dev) {
    const char* fn = "dcasgd_check_adaptive_lambda_grid";
    if (!mismatches_dev) return fail(DCASGD_EINVAL, "%s: mismatches_dev is NULL", fn);
    if (reinterpret_cast<uintptr_t>(mismatches_dev) & 7u) return fail(DCASGD_EALIGN, "%s: mismatches_dev must be 8-byte aligned", fn);
    if (a_count == 0) return DCASGD_OK;
    uint32_t a0, b0, b1;
    std::memcpy(&a0, &a_first, 4);
    const uint64_t a_last_bits = (uint64_t)a0 + (uint64_t)(a_count - 1) * a_step;
    if (a_last_bits > 0xFFFFFFFFull || ((uint32_t)a_last_bits ^ a0) >> 31) return fail(DCASGD_EINVAL, "%s: the numerators leave the sign's half of the encodings", fn);
    float a_last;
    const uint32_t al_bits = (uint32_t)a_last_bits;
    std::memcpy(&a_last, &al_bits, 4);
    const float lo = std::fabs(a_first), hi = std::fabs(a_last);      // bit patterns grow with the magnitude
    if (!(lo >= 0x1p-60f && hi < 0x1p60f)) return fail(DCASGD_EINVAL, "%s: every |a| must be in [2^-60, 2^60)", fn);
    if (!(s_first >= 0x1p-100f && s_last < 0x1p100f && s_first <= s_last))
        return fail(DCASGD_EINVAL, "%s: need 2^-100 <= s_first <= s_last < 2^100", fn);
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(fn, e);
    if (const int rc = check_device_buffer(fn, "mismatches_dev", mismatches_dev, 8, dev)) return rc;
    int sms = 148;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { (void)cudaGetLastError(); sms = 148; }
    std::memcpy(&b0, &s_first, 4);
    std::memcpy(&b1, &s_last, 4);
    const uint64_t s_count = (uint64_t)b1 - b0 + 1;
    // launches of bounded length: at most about 3e11 comparisons each (a fraction of a second)
    const uint64_t per = std::max<uint64_t>(1, std::min<uint64_t>(a_count, (300ull << 30) / s_count));
    const uint64_t pairs = (s_count + 1) / 2;
    const unsigned grid = (unsigned)std::min<uint64_t>((pairs + kThreads - 1) / kThreads, (uint64_t)sms * 64);
    // few radicands: spread the numerators over blockIdx.y until the GPU is full
    const unsigned grid_y = (unsigned)std::max<uint64_t>(1, std::min<uint64_t>({(uint64_t)sms * 8 / grid, (uint64_t)per, 4096}));
#ifdef DCASGD_DEBUG_CHECKS
    if (const int rc = debug_arm(static_cast<cudaStream_t>(stream), nullptr, g_default_debug_status, mismatches_dev, 8, true)) return rc;
#endif
    for (uint64_t done = 0; done < a_count; done += per) {
        const uint32_t na = (uint32_t)std::min<uint64_t>(per, a_count - done);
        k_check_lambda_grid<<<dim3(grid, grid_y), kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
            make_hyper(1.0f, 0.0f, 0.0f, 0.0f, kLambdaChecked), a0 + (uint32_t)(done * a_step), na, a_step, b0, s_count,
            reinterpret_cast<unsigned long long*>(mismatches_dev));
        e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail("lambda grid self-check kernel", e);
    }
    return DCASGD_OK;
}

int dcasgd_get_window_slot_cap(const dcasgd_server* s, uint32_t* max_slots) {
    if (!s || !max_slots) return fail(DCASGD_EINVAL, "dcasgd_get_window_slot_cap: NULL argument");
    *max_slots = s->slot_cap;
    return DCASGD_OK;
}

int dcasgd_debug_checks(dcasgd_server* s, uint32_t* status_dev) {
#ifdef DCASGD_DEBUG_CHECKS
    if (status_dev) {
        if (reinterpret_cast<uintptr_t>(status_dev) & 3u) return fail(DCASGD_EALIGN, "dcasgd_debug_checks: status_dev must be 4-byte aligned");
        int dev = -1;
        const cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return cuda_fail("dcasgd_debug_checks: cudaGetDevice", e);
        if (const int rc = check_device_buffer("dcasgd_debug_checks", "status_dev", status_dev, 4, dev)) return rc;
    }
    if (s) s->debug_status = status_dev;
    else g_default_debug_status = status_dev;
    return DCASGD_OK;
#else
    (void)s;
    (void)status_dev;
    return fail(DCASGD_EINVAL, "dcasgd_debug_checks: this library was built without -DDCASGD_DEBUG_CHECKS");
#endif
}

int dcasgd_get_launch_count(const dcasgd_server* s, uint64_t* launches) {
    if (!s || !launches) return fail(DCASGD_EINVAL, "dcasgd_get_launch_count: NULL argument");
    *launches = s->launches;
    return DCASGD_OK;
}

}  // extern "C"
