// Host side of the OD-SGD update library: context, validation, kernel selection
// and launches behind the C ABI declared in odsgd.h.  No torch types, no
// allocation of parameter-sized memory, no synchronisation.  The per-call path of the
// update entry points allocates nothing on the host either: buffers are enumerated into
// fixed arrays on the stack and error texts are only built when a call fails.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "odsgd.h"
#include "odsgd_kernels.cuh"

using namespace odsgd;

struct odsgd_ctx {
    int device = 0;
    int sm_count = 0;
    float* w[2] = {nullptr, nullptr};
    int cur = 0;  // index of the half that holds the current weights
    bool pingpong = false;
    float* w_delayed = nullptr;  // in-place layout: optional backup arena
    float* v = nullptr;          // NULL only in a worker-only context
    float* local[ODSGD_MAX_WORKERS] = {};
    float* mean_square[ODSGD_MAX_WORKERS] = {};
    size_t n = 0;
    std::vector<size_t> offsets;
    bool offsets_vec_ok = true;  // every tensor offset is a multiple of 4 elements
    int n_workers = 0;
    float lr = 0, local_lr = 0, momentum = 0, wd = 0;
    uint32_t flags = 0;
    int local_rule = ODSGD_LOCAL_SGD;
    float dc_lambda = 0, dc_m = 0, dc_eps = 0;
    const float* bound[ODSGD_MAX_WORKERS] = {};  // gradients of the latest global update
    bool grads_bound = false;
    const float* delayed = nullptr;  // weights from before the latest global update, if kept
    uint64_t step = 0;
    uint64_t launches = 0;
    int block_threads = 0;  // 0 = built-in
    int ctas_per_sm = 0;    // 0 = built-in
    // per-tensor multipliers: one device allocation [offsets u64 x (T+1) | lr_mult f32 x T | wd_mult f32 x T]
    void* table_dev = nullptr;
    std::vector<unsigned char> table_host;  // staging copy the upload reads from
    bool mult_on = false;
    float* server_ms = nullptr;  // Eq. 6 state of the server-side DC-ASGD step
    // weight mirrors: mirror[h][i] receives what the server kernel writes into weight half h
    float* mirror[2][ODSGD_MAX_MIRRORS] = {};
    int n_mirrors = 0;
    uint64_t wp = 0;             // Algorithm 2's warm-up length
    uint64_t iter = 0;           // iterations done through odsgd_step
    // host-buffer entry point with a separate copy stream: ordering between the two streams
    cudaEvent_t ev_kernel_done = nullptr;  // recorded on the compute stream after the update kernel
    cudaEvent_t ev_copy_done = nullptr;    // recorded on the copy stream after the device-to-host copy
    bool copy_pending = false;             // ev_copy_done guards a copy-back no later kernel may overtake
    bool copy_waited = false;              // a stream has been made to wait for that copy already ...
    cudaStream_t copy_waited_on = nullptr; // ... this one: work enqueued on it later is ordered behind the copy
    // gradient tables checked once by odsgd_bind_grads
    struct Binding {
        bool used = false;
        uint64_t epoch = 0;  // state_epoch at the time the table was checked
        const float* g[ODSGD_MAX_WORKERS] = {};
    };
    Binding bindings[ODSGD_MAX_BINDINGS];
    uint64_t state_epoch = 0;  // bumped whenever the set of state buffers changes
    // resident CTAs per SM by (kernel, block size); 0 = that block size cannot be launched
    std::map<std::pair<const void*, int>, int> occupancy;
    std::string err;
};

namespace {

thread_local std::string g_create_err;

int fail(odsgd_ctx* ctx, int code, const std::string& msg) {
    if (ctx) ctx->err = msg; else g_create_err = msg;
    return code;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

bool overlap(const void* a, const void* b, size_t bytes) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + bytes && y < x + bytes;
}

struct Named {
    const void* p;
    const char* name;
    int idx;
};

std::string label(const Named& b) {
    char buf[64];
    if (b.idx >= 0) snprintf(buf, sizeof buf, "%s[%d]", b.name, b.idx); else snprintf(buf, sizeof buf, "%s", b.name);
    return buf;
}

// A short list of named buffers on the stack (no heap traffic on the per-call path).
template <int CAP>
struct BufList {
    Named b[CAP];
    int n = 0;
    void add(const void* p, const char* name, int idx) {
        if (n < CAP) b[n++] = Named{p, name, idx};
    }
};
constexpr int kMaxState = 5 + 2 * ODSGD_MAX_WORKERS + 2 * ODSGD_MAX_MIRRORS;
using StateList = BufList<kMaxState>;
using CallList = BufList<kMaxState + ODSGD_MAX_WORKERS + 4>;

// State buffers of a context, for alias checks.
void state_buffers(const odsgd_ctx* c, StateList* s) {
    s->n = 0;
    s->add(c->w[0], "w_a", -1);
    if (c->w[1]) s->add(c->w[1], "w_b", -1);
    if (c->w_delayed) s->add(c->w_delayed, "w_delayed", -1);
    if (c->v) s->add(c->v, "v", -1);
    for (int m = 0; m < c->n_workers; ++m) {
        if (c->local[m]) s->add(c->local[m], "local", m);
        if (c->mean_square[m]) s->add(c->mean_square[m], "mean_square", m);
    }
    if (c->server_ms) s->add(c->server_ms, "server_mean_square", -1);
    for (int i = 0; i < c->n_mirrors; ++i) {
        s->add(c->mirror[0][i], "mirrors_a", i);
        if (c->mirror[1][i]) s->add(c->mirror[1][i], "mirrors_b", i);
    }
}

int check_distinct(odsgd_ctx* err_ctx, const StateList& s, size_t bytes) {
    for (int i = 0; i < s.n; ++i)
        for (int j = i + 1; j < s.n; ++j)
            if (overlap(s.b[i].p, s.b[j].p, bytes))
                return fail(err_ctx, ODSGD_ERR_OVERLAP, label(s.b[i]) + " overlaps " + label(s.b[j]));
    return ODSGD_OK;
}

// One outside buffer (a gradient, a caller-supplied backup) against the context's state.
int check_outside(odsgd_ctx* c, const StateList& st, const Named& g) {
    const size_t bytes = c->n * sizeof(float);
    for (int i = 0; i < st.n; ++i)
        if (overlap(g.p, st.b[i].p, bytes)) return fail(c, ODSGD_ERR_OVERLAP, label(g) + " overlaps " + label(st.b[i]));
    return ODSGD_OK;
}

// Vector width usable for a call: 4 lanes when every pointer it touches is 16-byte aligned,
// else 1 lane if the context allows it.  Returns 0 and sets the error otherwise.  The common
// case is decided from the OR of all addresses; the buffers are only walked by name to word
// the error.
template <int CAP>
int lanes_for(odsgd_ctx* c, const BufList<CAP>& ptrs) {
    uintptr_t bits = 0;
    for (int i = 0; i < ptrs.n; ++i) bits |= reinterpret_cast<uintptr_t>(ptrs.b[i].p);
    if ((bits & 15) == 0) return 4;
    const bool scalar_ok = (c->flags & ODSGD_FLAG_ALLOW_UNALIGNED) != 0;
    if ((bits & 3) == 0 && scalar_ok) return 1;
    for (int i = 0; i < ptrs.n; ++i) {
        const Named& b = ptrs.b[i];
        if (!aligned(b.p, 4)) {
            fail(c, ODSGD_ERR_ALIGN, label(b) + " is not 4-byte aligned");
            return 0;
        }
        if (!aligned(b.p, 16) && !scalar_ok) {
            fail(c, ODSGD_ERR_ALIGN, label(b) + " is not 16-byte aligned (set ODSGD_FLAG_ALLOW_UNALIGNED for the scalar path)");
            return 0;
        }
    }
    return 1;
}

int grid_for(const odsgd_ctx* c, unsigned long long n, int lanes, int block, int per_thread, int resident_default) {
    const unsigned long long nvec = n / lanes > 0 ? n / lanes : 1;
    const unsigned long long tile = (unsigned long long)block * per_thread;
    const unsigned long long tiles = (nvec + tile - 1) / tile;
    const int per_sm = c->ctas_per_sm > 0 ? c->ctas_per_sm : resident_default;
    const unsigned long long cap = (unsigned long long)c->sm_count * per_sm;
    return (int)(tiles < cap ? tiles : cap);
}

int after_launch(odsgd_ctx* c, const char* what) {
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
    c->launches += 1;
    return ODSGD_OK;
}

// Resident CTAs per SM for a kernel at a block size; 0 when the kernel cannot be launched
// with that many threads (register file too small).
template <typename K>
int resident_ctas(K kernel, int block) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, block, 0) != cudaSuccess || n < 1) {
        cudaGetLastError();
        n = 0;
    }
    return n;
}

// Cached per context (a context belongs to one device and is used from one thread at a time).
template <typename K>
int resident_cached(odsgd_ctx* c, K kernel, int block) {
    const std::pair<const void*, int> key(reinterpret_cast<const void*>(kernel), block);
    auto it = c->occupancy.find(key);
    if (it != c->occupancy.end()) return it->second;
    const int n = resident_ctas(kernel, block);
    c->occupancy[key] = n;
    return n;
}

// Every launching call runs on the device the context was created on.
int on_own_device(odsgd_ctx* c) {
    int dev = -1;
    const cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
    if (dev != c->device)
        return fail(c, ODSGD_ERR_STATE, "the current CUDA device (" + std::to_string(dev) + ") is not the one the context was created on (" +
                                            std::to_string(c->device) + ")");
    return ODSGD_OK;
}

// One launch on `st`, marked so that it may be scheduled while the kernel ahead of it in the
// stream is still draining (the kernels themselves wait for that kernel's completion before
// they touch memory).
template <typename Args>
void launch_kernel(void (*kernel)(const Args), int grid, int block, cudaStream_t st, const Args& a) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3((unsigned)block, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = kProgrammaticLaunch ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, a);  // the error, if any, is picked up by after_launch
}

int too_wide(odsgd_ctx* c, int block) {
    return fail(c, ODSGD_ERR_UNSUPPORTED, "block_threads = " + std::to_string(block) + " is too large for this kernel");
}

// `dry`: stop after the checks that can still refuse the launch (block size against the
// kernel's register use), so that a caller can validate everything before it enqueues copies.
template <bool DET, int NL, int LOCAL, int RULE, bool MULT, int BB, int UB>
int launch_server_k(odsgd_ctx* c, const ServerArgs& a, cudaStream_t st, bool dry) {
    const int block = c->block_threads > 0 ? c->block_threads : server_default_block(LOCAL, RULE);
    auto kernel = server_kernel<DET, NL, LOCAL, RULE, MULT, BB, UB>;
    if (resident_cached(c, kernel, block) == 0) return too_wide(c, block);
    if (dry) return ODSGD_OK;
    const int grid = grid_for(c, a.n, NL, block, server_vectors_per_thread(LOCAL, RULE, UB), server_grid_cap(a.n_workers));
    launch_kernel<ServerArgs>(kernel, grid, block, st, a);
    return after_launch(c, "server kernel launch");
}

template <bool DET, int NL, int LOCAL, int RULE, bool MULT>
int launch_server_m(odsgd_ctx* c, const ServerArgs& a, cudaStream_t st, bool dry) {
    // the shape follows the worker count on the 128-bit path; the scalar fallback and the
    // all-workers variants (whose shape is fixed inside the kernel) keep a single instantiation
    if constexpr (LOCAL == kLocalOne && NL == 4 && needs_prev(RULE) && needs_state(RULE)) {
        // one worker's Eq. 5-6 update carries two more vectors per tile vector than the other
        // rules (previous local weights and mean square): the wide few-worker shapes spill and
        // the narrower ones win (2 x 3 against 2 x 4: +15-18 % at M <= 2, +3 % at M = 4; 8 x 2
        // against 3 x 4 / 4 x 3: +6 % at M = 6, +4 % at M = 8, +1 % at M = 12)
        if (a.n_workers <= 4) return launch_server_k<DET, NL, LOCAL, RULE, MULT, 2, 3>(c, a, st, dry);
    } else if constexpr (LOCAL != kLocalAll && NL == 4) {
        switch (server_shape_for(a.n_workers)) {
            case kShape2x4: return launch_server_k<DET, NL, LOCAL, RULE, MULT, ODSGD_SHAPE0_B, ODSGD_SHAPE0_U>(c, a, st, dry);
            case kShape3x4:
                // 3 x 4 fits the register budget only without a state arena or a multiplier
                // lookup in the tile; the variants that have one take 4 x 3 (no spills)
                if constexpr (!MULT && !needs_state(RULE))
                    return launch_server_k<DET, NL, LOCAL, RULE, MULT, ODSGD_SHAPE1_B, ODSGD_SHAPE1_U>(c, a, st, dry);
                else
                    return launch_server_k<DET, NL, LOCAL, RULE, MULT, ODSGD_SHAPE2_B, ODSGD_SHAPE2_U>(c, a, st, dry);
            case kShape4x3: return launch_server_k<DET, NL, LOCAL, RULE, MULT, ODSGD_SHAPE2_B, ODSGD_SHAPE2_U>(c, a, st, dry);
            default: break;
        }
    }
    return launch_server_k<DET, NL, LOCAL, RULE, MULT, kBatch, kUnroll>(c, a, st, dry);
}

template <bool DET, int NL, int LOCAL, int RULE>
int launch_server_t(odsgd_ctx* c, const ServerArgs& a, bool mult, cudaStream_t st, bool dry) {
    return mult ? launch_server_m<DET, NL, LOCAL, RULE, true>(c, a, st, dry)
                : launch_server_m<DET, NL, LOCAL, RULE, false>(c, a, st, dry);
}

template <bool DET, int NL, int LOCAL>
int launch_server_r(odsgd_ctx* c, const ServerArgs& a, bool mult, cudaStream_t st, bool dry) {
    if constexpr (LOCAL == kLocalNone || LOCAL == kLocalNoneMirrored) {
        return launch_server_t<DET, NL, LOCAL, ODSGD_LOCAL_SGD>(c, a, mult, st, dry);
    } else {
        switch (c->local_rule) {
            case ODSGD_LOCAL_SGD: return launch_server_t<DET, NL, LOCAL, ODSGD_LOCAL_SGD>(c, a, mult, st, dry);
            case ODSGD_LOCAL_DC_C: return launch_server_t<DET, NL, LOCAL, ODSGD_LOCAL_DC_C>(c, a, mult, st, dry);
            case ODSGD_LOCAL_MOMENTUM: return launch_server_t<DET, NL, LOCAL, ODSGD_LOCAL_MOMENTUM>(c, a, mult, st, dry);
            default: return launch_server_t<DET, NL, LOCAL, ODSGD_LOCAL_DC_A>(c, a, mult, st, dry);
        }
    }
}

template <bool DET, int NL>
int launch_server_l(odsgd_ctx* c, const ServerArgs& a, int local_mode, bool mult, cudaStream_t st, bool dry) {
    switch (local_mode) {
        case kLocalNone: return launch_server_r<DET, NL, kLocalNone>(c, a, mult, st, dry);
        case kLocalOne: return launch_server_r<DET, NL, kLocalOne>(c, a, mult, st, dry);
        case kLocalNoneMirrored: return launch_server_r<DET, NL, kLocalNoneMirrored>(c, a, mult, st, dry);
        default: return launch_server_r<DET, NL, kLocalAll>(c, a, mult, st, dry);
    }
}

int launch_server(odsgd_ctx* c, const ServerArgs& a, int lanes, int local_mode, bool mult, cudaStream_t st, bool dry) {
    const bool det = (c->flags & ODSGD_FLAG_ALLOW_FMA) == 0;
    if (det)
        return lanes == 4 ? launch_server_l<true, 4>(c, a, local_mode, mult, st, dry)
                          : launch_server_l<true, 1>(c, a, local_mode, mult, st, dry);
    return lanes == 4 ? launch_server_l<false, 4>(c, a, local_mode, mult, st, dry)
                      : launch_server_l<false, 1>(c, a, local_mode, mult, st, dry);
}

template <bool DET, int NL, int RULE, bool SERVER>
int launch_local_t(odsgd_ctx* c, const LocalArgs& a, cudaStream_t st) {
    const int block = c->block_threads > 0 ? c->block_threads : local_default_block(RULE);
    auto kernel = local_kernel<DET, NL, RULE, SERVER>;
    if (resident_cached(c, kernel, block) == 0) return too_wide(c, block);
    launch_kernel<LocalArgs>(kernel, grid_for(c, a.n, NL, block, kLocalUnroll, kLocalCtasPerSm), block, st, a);
    return after_launch(c, "local kernel launch");
}

template <bool DET, int NL>
int launch_local_r(odsgd_ctx* c, const LocalArgs& a, bool server, cudaStream_t st) {
    if (server) {  // DC-ASGD at the server: only the delay-compensated rules exist there
        return c->local_rule == ODSGD_LOCAL_DC_C ? launch_local_t<DET, NL, ODSGD_LOCAL_DC_C, true>(c, a, st)
                                                 : launch_local_t<DET, NL, ODSGD_LOCAL_DC_A, true>(c, a, st);
    }
    switch (c->local_rule) {
        case ODSGD_LOCAL_SGD: return launch_local_t<DET, NL, ODSGD_LOCAL_SGD, false>(c, a, st);
        case ODSGD_LOCAL_DC_C: return launch_local_t<DET, NL, ODSGD_LOCAL_DC_C, false>(c, a, st);
        case ODSGD_LOCAL_MOMENTUM: return launch_local_t<DET, NL, ODSGD_LOCAL_MOMENTUM, false>(c, a, st);
        default: return launch_local_t<DET, NL, ODSGD_LOCAL_DC_A, false>(c, a, st);
    }
}

int launch_local(odsgd_ctx* c, const LocalArgs& a, int lanes, bool server, cudaStream_t st) {
    const bool det = (c->flags & ODSGD_FLAG_ALLOW_FMA) == 0;
    if (det) return lanes == 4 ? launch_local_r<true, 4>(c, a, server, st) : launch_local_r<true, 1>(c, a, server, st);
    return lanes == 4 ? launch_local_r<false, 4>(c, a, server, st) : launch_local_r<false, 1>(c, a, server, st);
}

template <bool DET, int NL>
int launch_asgd_t(odsgd_ctx* c, const AsgdArgs& a, cudaStream_t st) {
    const int block = c->block_threads > 0 ? c->block_threads : kDefaultAsgdBlock;
    auto kernel = asgd_kernel<DET, NL>;
    if (resident_cached(c, kernel, block) == 0) return too_wide(c, block);
    launch_kernel<AsgdArgs>(kernel, grid_for(c, a.n, NL, block, kSmallUnroll, kAsgdCtasPerSm), block, st, a);
    return after_launch(c, "asgd kernel launch");
}

int launch_asgd(odsgd_ctx* c, const AsgdArgs& a, int lanes, cudaStream_t st) {
    const bool det = (c->flags & ODSGD_FLAG_ALLOW_FMA) == 0;
    if (det) return lanes == 4 ? launch_asgd_t<true, 4>(c, a, st) : launch_asgd_t<true, 1>(c, a, st);
    return lanes == 4 ? launch_asgd_t<false, 4>(c, a, st) : launch_asgd_t<false, 1>(c, a, st);
}

LocalParams local_params(const odsgd_ctx* c) {
    LocalParams p;
    p.local_lr = c->local_lr;
    p.lambda = c->dc_lambda;
    p.m = c->dc_m;
    p.one_minus_m = 1.0f - c->dc_m;
    p.eps = c->dc_eps;
    p.first = 0;
    return p;
}

// Run before every kernel that may write a local arena: the context's device must be
// current, and a copy-back of local weights that odsgd_fused_update_host put on a separate
// copy stream must be out before the kernel overwrites that arena.  Every stream that comes
// by is made to wait for the copy (work behind it on the same stream is ordered anyway); the
// guard stays up until a later host-buffer call records a newer copy.
int before_launch(odsgd_ctx* c, cudaStream_t st) {
    const int rc_dev = on_own_device(c);
    if (rc_dev != ODSGD_OK) return rc_dev;
    if (!c->copy_pending) return ODSGD_OK;
    if (c->copy_waited && c->copy_waited_on == st) return ODSGD_OK;
    const cudaError_t e = cudaStreamWaitEvent(st, c->ev_copy_done, 0);
    if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("stream wait: ") + cudaGetErrorString(e));
    c->copy_waited = true;
    c->copy_waited_on = st;
    return ODSGD_OK;
}

// Checks a table of gradient pointers against the context's state buffers.
int check_grads(odsgd_ctx* c, const float* const* grads) {
    if (!grads) return fail(c, ODSGD_ERR_ARG, "worker_grads is NULL");
    StateList st;
    state_buffers(c, &st);
    for (int m = 0; m < c->n_workers; ++m) {
        if (!grads[m]) return fail(c, ODSGD_ERR_ARG, "worker_grads[" + std::to_string(m) + "] is NULL");
        const int rc = check_outside(c, st, Named{grads[m], "worker_grads", m});
        if (rc != ODSGD_OK) return rc;
    }
    return ODSGD_OK;
}

// A fully validated server-kernel launch: arguments, vector width, and what the context's
// state becomes once the launch is in the stream.
struct ServerPlan {
    ServerArgs a;
    int lanes = 0;
    int local_mode = kLocalNone;
    bool mult = false;
    bool keep_backup = false;
    int next_cur = 0;
    const float* delayed_after = nullptr;
};

// Local mode and outputs for a fused call; fills a.x / a.ms / a.local_worker.
int bind_local_outputs(odsgd_ctx* c, int worker_id, ServerArgs* a, int* local_mode, CallList* ptrs) {
    if (worker_id >= c->n_workers || worker_id < -1) return fail(c, ODSGD_ERR_ARG, "worker_id out of range");
    const bool need_ms = needs_state(c->local_rule);
    if (worker_id >= 0) {
        if (!c->local[worker_id]) return fail(c, ODSGD_ERR_ARG, "no local buffer for worker " + std::to_string(worker_id));
        if (need_ms && !c->mean_square[worker_id]) return fail(c, ODSGD_ERR_STATE, "no mean-square arena for that worker");
        a->x[0] = c->local[worker_id];
        a->ms[0] = c->mean_square[worker_id];
        a->local_worker = worker_id;
        ptrs->add(a->x[0], "local", worker_id);
        if (need_ms) ptrs->add(a->ms[0], "mean_square", worker_id);
        *local_mode = kLocalOne;
        return ODSGD_OK;
    }
    int count = 0;
    for (int m = 0; m < c->n_workers; ++m) {
        a->x[m] = c->local[m];
        a->ms[m] = c->mean_square[m];
        if (c->local[m]) {
            if (need_ms && !c->mean_square[m]) return fail(c, ODSGD_ERR_STATE, "no mean-square arena for worker " + std::to_string(m));
            ptrs->add(a->x[m], "local", m);
            if (need_ms) ptrs->add(a->ms[m], "mean_square", m);
            ++count;
        }
    }
    if (count == 0) return fail(c, ODSGD_ERR_ARG, "worker_id == -1 but the context has no local buffers");
    *local_mode = kLocalAll;
    return ODSGD_OK;
}

// Builds the plan of a global, fused or SSGD call from a gradient table that has already been
// checked against the state buffers (check_grads, at call or at bind time).
//   keep_backup:  OD-SGD server step (the old weights stay available to the workers)
//   local_id:     -2 none, -1 all workers, >= 0 one worker
//   static_table: device address of a multiplier table to use instead of the context's own
int plan_server(odsgd_ctx* c, const float* const* grads, bool keep_backup, int local_id, bool first_delayed_step,
                const unsigned char* static_table, ServerPlan* p) {
    if (!c->v) return fail(c, ODSGD_ERR_STATE, "a worker-only context (ODSGD_FLAG_WORKER_ONLY) has no server state");
    ServerArgs& a = p->a;
    memset(&a, 0, sizeof a);
    CallList ptrs;
    for (int m = 0; m < c->n_workers; ++m) {
        a.g[m] = grads[m];
        ptrs.add(grads[m], "worker_grads", m);
    }
    a.v = c->v;
    a.n = c->n;
    a.n_workers = c->n_workers;
    a.inv_n = 1.0f / (float)c->n_workers;
    a.lr = c->lr;
    a.momentum = c->momentum;
    a.wd = c->wd;
    a.lp = local_params(c);
    a.lp.first = first_delayed_step ? 1 : 0;
    p->mult = static_table != nullptr || c->mult_on;
    if (p->mult) {
        const size_t nt = c->offsets.size() - 1;
        const unsigned char* base = static_table ? static_table : static_cast<const unsigned char*>(c->table_dev);
        a.t_off = reinterpret_cast<const unsigned long long*>(base);
        a.t_lr_mult = reinterpret_cast<const float*>(base + (nt + 1) * sizeof(unsigned long long));
        a.t_wd_mult = a.t_lr_mult + nt;
        a.n_tensors = (unsigned int)nt;
    }
    a.w_in = c->w[c->cur];
    p->keep_backup = keep_backup;
    p->delayed_after = nullptr;
    p->next_cur = c->cur;
    if (keep_backup && c->pingpong) {
        a.w_out = c->w[c->cur ^ 1];
        p->delayed_after = c->w[c->cur];
        p->next_cur = c->cur ^ 1;
    } else {
        a.w_out = c->w[c->cur];
        if (keep_backup && c->w_delayed) {
            a.w_prev = c->w_delayed;
            p->delayed_after = c->w_delayed;
        }
    }
    ptrs.add(a.w_in, "w", -1);
    ptrs.add(a.w_out, "w", -1);
    ptrs.add(a.v, "v", -1);
    if (a.w_prev) ptrs.add(a.w_prev, "w_delayed", -1);

    p->local_mode = kLocalNone;
    if (c->n_mirrors > 0) {
        // only the plain server pass keeps mirrors in step with the weights
        if (local_id >= -1)
            return fail(c, ODSGD_ERR_STATE, "weight mirrors are set: only odsgd_global_update / odsgd_ssgd_step (and their bound forms) can run");
        const int half = a.w_out == c->w[1] ? 1 : 0;
        for (int i = 0; i < c->n_mirrors; ++i) {
            a.w_mirror[i] = c->mirror[half][i];
            ptrs.add(a.w_mirror[i], half ? "mirrors_b" : "mirrors_a", i);
        }
        a.n_mirrors = c->n_mirrors;
        p->local_mode = kLocalNoneMirrored;
    }
    if (local_id >= -1) {
        const int rc = bind_local_outputs(c, local_id, &a, &p->local_mode, &ptrs);
        if (rc != ODSGD_OK) return rc;
    }
    p->lanes = lanes_for(c, ptrs);
    if (p->lanes == 0) return ODSGD_ERR_ALIGN;
    // with multipliers a 128-bit vector must not straddle two tensors (the calls that switch
    // them on have checked that the scalar path is allowed when it would)
    if (p->mult && p->lanes == 4 && !c->offsets_vec_ok) p->lanes = 1;
    return ODSGD_OK;
}

// Launches a plan (or, with dry = true, only runs the checks that could still refuse it)
// and moves the context's state on.
int run_server(odsgd_ctx* c, const ServerPlan& p, cudaStream_t st, bool dry) {
    int rc = dry ? on_own_device(c) : before_launch(c, st);
    if (rc != ODSGD_OK) return rc;
    rc = launch_server(c, p.a, p.lanes, p.local_mode, p.mult, st, dry);
    if (rc != ODSGD_OK || dry) return rc;
    c->cur = p.next_cur;
    c->step += 1;
    c->delayed = p.delayed_after;
    c->grads_bound = p.keep_backup;
    if (p.keep_backup)
        for (int m = 0; m < c->n_workers; ++m) c->bound[m] = p.a.g[m];
    return ODSGD_OK;
}

// Shared body of the global, fused and SSGD calls on an unchecked gradient table.
int server_call(odsgd_ctx* c, const float* const* grads, bool keep_backup, int local_id, void* stream,
                bool first_delayed_step = false) {
    if (!c) return ODSGD_ERR_ARG;
    int rc = check_grads(c, grads);
    if (rc != ODSGD_OK) return rc;
    ServerPlan p;
    rc = plan_server(c, grads, keep_backup, local_id, first_delayed_step, nullptr, &p);
    if (rc != ODSGD_OK) return rc;
    return run_server(c, p, static_cast<cudaStream_t>(stream), false);
}

// The same on a table odsgd_bind_grads has checked: no scan of the state buffers.
int bound_call(odsgd_ctx* c, int slot, bool keep_backup, int local_id, void* stream, bool first_delayed_step = false) {
    if (!c) return ODSGD_ERR_ARG;
    if (slot < 0 || slot >= ODSGD_MAX_BINDINGS || !c->bindings[slot].used)
        return fail(c, ODSGD_ERR_ARG, "no gradient table is bound to slot " + std::to_string(slot));
    const odsgd_ctx::Binding& b = c->bindings[slot];
    if (b.epoch != c->state_epoch)
        return fail(c, ODSGD_ERR_STATE, "the context's buffers changed after slot " + std::to_string(slot) +
                                            " was bound: bind the gradient table again");
    ServerPlan p;
    const int rc = plan_server(c, b.g, keep_backup, local_id, first_delayed_step, nullptr, &p);
    if (rc != ODSGD_OK) return rc;
    return run_server(c, p, static_cast<cudaStream_t>(stream), false);
}

// Algorithm 2's schedule: which server call iteration c->iter is.
template <typename F>
int scheduled_step(odsgd_ctx* c, F call) {
    int rc;
    if (c->iter < c->wp) {
        rc = call(false, -2, false);  // warm-up stage: SSGD
    } else {
        // from the last warm-up iteration on: server step + local update of every worker; at
        // iteration wp itself the gradients were taken on the global weights (no delay yet)
        rc = call(true, -1, c->iter == c->wp);
    }
    if (rc == ODSGD_OK) c->iter += 1;
    return rc;
}

}  // namespace

extern "C" {

int odsgd_version(void) { return ODSGD_VERSION_MAJOR * 1000 + ODSGD_VERSION_MINOR; }

const char* odsgd_strerror(int code) {
    switch (code) {
        case ODSGD_OK: return "ok";
        case ODSGD_ERR_ARG: return "invalid argument";
        case ODSGD_ERR_ALIGN: return "misaligned device pointer";
        case ODSGD_ERR_OVERLAP: return "buffers overlap";
        case ODSGD_ERR_STATE: return "call not valid in this state";
        case ODSGD_ERR_CUDA: return "CUDA error";
        case ODSGD_ERR_UNSUPPORTED: return "not supported";
        default: return "unknown error code";
    }
}

int odsgd_create(odsgd_ctx** out, const odsgd_desc* d) {
    if (!out) return fail(nullptr, ODSGD_ERR_ARG, "out is NULL");
    *out = nullptr;
    if (!d) return fail(nullptr, ODSGD_ERR_ARG, "desc is NULL");
    constexpr uint32_t known =
        ODSGD_FLAG_DETERMINISTIC | ODSGD_FLAG_ALLOW_UNALIGNED | ODSGD_FLAG_ALLOW_FMA | ODSGD_FLAG_WORKER_ONLY;
    const bool worker_only = (d->flags & ODSGD_FLAG_WORKER_ONLY) != 0;
    if (!d->w_a || (!d->v && !worker_only)) return fail(nullptr, ODSGD_ERR_ARG, "w_a and v must not be NULL");
    if (d->n_params == 0) return fail(nullptr, ODSGD_ERR_ARG, "n_params is 0");
    if (d->n_workers < 1 || d->n_workers > ODSGD_MAX_WORKERS)
        return fail(nullptr, ODSGD_ERR_ARG, "n_workers must be in 1.." + std::to_string(ODSGD_MAX_WORKERS));
    if (d->w_b && d->w_delayed) return fail(nullptr, ODSGD_ERR_ARG, "w_delayed must be NULL in the ping-pong layout");
    if (!d->tensor_offsets || d->n_tensors < 1) return fail(nullptr, ODSGD_ERR_ARG, "tensor_offsets / n_tensors missing");
    if (d->tensor_offsets[0] != 0 || d->tensor_offsets[d->n_tensors] != d->n_params)
        return fail(nullptr, ODSGD_ERR_ARG, "tensor_offsets must start at 0 and end at n_params");
    for (size_t t = 0; t < d->n_tensors; ++t)
        if (d->tensor_offsets[t + 1] <= d->tensor_offsets[t])
            return fail(nullptr, ODSGD_ERR_ARG, "tensor_offsets must be strictly ascending (at tensor " + std::to_string(t) + ")");
    if (d->flags & ~known) return fail(nullptr, ODSGD_ERR_ARG, "unknown flag bits");
    if ((d->flags & ODSGD_FLAG_DETERMINISTIC) && (d->flags & ODSGD_FLAG_ALLOW_FMA))
        return fail(nullptr, ODSGD_ERR_ARG, "ODSGD_FLAG_DETERMINISTIC and ODSGD_FLAG_ALLOW_FMA exclude each other");

    odsgd_ctx* c = new (std::nothrow) odsgd_ctx;
    if (!c) return fail(nullptr, ODSGD_ERR_ARG, "out of host memory");
    c->w[0] = d->w_a;
    c->w[1] = d->w_b;
    c->pingpong = d->w_b != nullptr;
    c->w_delayed = d->w_delayed;
    c->v = d->v;
    c->n = d->n_params;
    c->n_workers = d->n_workers;
    c->offsets.assign(d->tensor_offsets, d->tensor_offsets + d->n_tensors + 1);
    for (size_t o : c->offsets)
        if (o % 4 != 0) c->offsets_vec_ok = false;
    c->lr = d->lr;
    c->local_lr = d->local_lr;
    c->momentum = d->momentum;
    c->wd = d->wd;
    c->flags = d->flags;
    if (d->local)
        for (int m = 0; m < d->n_workers; ++m) c->local[m] = d->local[m];

    StateList st;
    state_buffers(c, &st);
    const size_t need = (d->flags & ODSGD_FLAG_ALLOW_UNALIGNED) ? 4 : 16;
    for (int i = 0; i < st.n; ++i) {
        if (!aligned(st.b[i].p, need)) {
            const std::string msg = label(st.b[i]) + " is not " + std::to_string(need) + "-byte aligned";
            delete c;
            return fail(nullptr, ODSGD_ERR_ALIGN, msg);
        }
    }
    int rc = check_distinct(nullptr, st, c->n * sizeof(float));
    if (rc != ODSGD_OK) {
        delete c;
        return rc;
    }
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    if (e != cudaSuccess || c->sm_count < 1) {
        const std::string msg = std::string("no usable CUDA device: ") + cudaGetErrorString(e);
        cudaGetLastError();
        delete c;
        return fail(nullptr, ODSGD_ERR_CUDA, msg);
    }
    *out = c;
    return ODSGD_OK;
}

int odsgd_destroy(odsgd_ctx* ctx) {
    if (!ctx) return ODSGD_ERR_ARG;
    if (ctx->table_dev) cudaFree(ctx->table_dev);
    if (ctx->ev_kernel_done) cudaEventDestroy(ctx->ev_kernel_done);
    if (ctx->ev_copy_done) cudaEventDestroy(ctx->ev_copy_done);
    delete ctx;
    return ODSGD_OK;
}

int odsgd_global_update(odsgd_ctx* ctx, const float* const* worker_grads, void* stream) {
    return server_call(ctx, worker_grads, true, -2, stream);
}

int odsgd_fused_update(odsgd_ctx* ctx, const float* const* worker_grads, int worker_id, void* stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    if (worker_id < -1 || worker_id >= ctx->n_workers) return fail(ctx, ODSGD_ERR_ARG, "worker_id out of range");
    return server_call(ctx, worker_grads, true, worker_id, stream);
}

int odsgd_ssgd_step(odsgd_ctx* ctx, const float* const* worker_grads, void* stream) {
    return server_call(ctx, worker_grads, false, -2, stream);
}

int odsgd_bind_grads(odsgd_ctx* ctx, const float* const* worker_grads, int* slot) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    if (!slot) return fail(c, ODSGD_ERR_ARG, "slot is NULL");
    *slot = -1;
    int rc = check_grads(c, worker_grads);
    if (rc != ODSGD_OK) return rc;
    // alignment is a property of the table too: refuse now what every later call would refuse
    CallList ptrs;
    for (int m = 0; m < c->n_workers; ++m) ptrs.add(worker_grads[m], "worker_grads", m);
    if (lanes_for(c, ptrs) == 0) return ODSGD_ERR_ALIGN;
    for (int s = 0; s < ODSGD_MAX_BINDINGS; ++s) {
        odsgd_ctx::Binding& b = c->bindings[s];
        if (b.used) continue;
        b.used = true;
        b.epoch = c->state_epoch;
        for (int m = 0; m < ODSGD_MAX_WORKERS; ++m) b.g[m] = m < c->n_workers ? worker_grads[m] : nullptr;
        *slot = s;
        return ODSGD_OK;
    }
    return fail(c, ODSGD_ERR_UNSUPPORTED,
                "all " + std::to_string(ODSGD_MAX_BINDINGS) + " binding slots are in use (odsgd_unbind_grads frees one)");
}

int odsgd_unbind_grads(odsgd_ctx* ctx, int slot) {
    if (!ctx) return ODSGD_ERR_ARG;
    if (slot < 0 || slot >= ODSGD_MAX_BINDINGS || !ctx->bindings[slot].used)
        return fail(ctx, ODSGD_ERR_ARG, "no gradient table is bound to slot " + std::to_string(slot));
    ctx->bindings[slot].used = false;
    return ODSGD_OK;
}

int odsgd_global_update_bound(odsgd_ctx* ctx, int slot, void* stream) { return bound_call(ctx, slot, true, -2, stream); }

int odsgd_fused_update_bound(odsgd_ctx* ctx, int slot, int worker_id, void* stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    if (worker_id < -1 || worker_id >= ctx->n_workers) return fail(ctx, ODSGD_ERR_ARG, "worker_id out of range");
    return bound_call(ctx, slot, true, worker_id, stream);
}

int odsgd_ssgd_step_bound(odsgd_ctx* ctx, int slot, void* stream) { return bound_call(ctx, slot, false, -2, stream); }

int odsgd_local_update(odsgd_ctx* ctx, int worker_id, void* stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    if (worker_id < 0 || worker_id >= c->n_workers) return fail(c, ODSGD_ERR_ARG, "worker_id out of range");
    if (!c->grads_bound) return fail(c, ODSGD_ERR_STATE, "no gradients bound: call odsgd_global_update first");
    if (!c->delayed) return fail(c, ODSGD_ERR_STATE, "this context keeps no backup weights (in-place layout without w_delayed)");
    if (!c->local[worker_id]) return fail(c, ODSGD_ERR_ARG, "no local buffer for worker " + std::to_string(worker_id));
    const bool need_ms = needs_state(c->local_rule);
    if (need_ms && !c->mean_square[worker_id]) return fail(c, ODSGD_ERR_STATE, "no state arena (mean square / velocity) for that worker");
    LocalArgs a;
    a.w_bak = c->delayed;
    a.g = c->bound[worker_id];
    a.x = c->local[worker_id];
    a.ms = c->mean_square[worker_id];
    a.w_out = nullptr;
    a.n = c->n;
    a.lp = local_params(c);
    BufList<4> ptrs;
    ptrs.add(a.w_bak, "w_delayed", -1);
    ptrs.add(a.g, "worker_grads", worker_id);
    ptrs.add(a.x, "local", worker_id);
    if (need_ms) ptrs.add(a.ms, "mean_square", worker_id);
    const int lanes = lanes_for(c, ptrs);
    if (lanes == 0) return ODSGD_ERR_ALIGN;
    const int rc_copy = before_launch(c, static_cast<cudaStream_t>(stream));
    if (rc_copy != ODSGD_OK) return rc_copy;
    return launch_local(c, a, lanes, false, static_cast<cudaStream_t>(stream));
}

int odsgd_worker_local_update(odsgd_ctx* ctx, int worker_id, const float* w_bak, const float* grad, int no_delay,
                              void* stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    if (worker_id < 0 || worker_id >= c->n_workers) return fail(c, ODSGD_ERR_ARG, "worker_id out of range");
    if (!w_bak || !grad) return fail(c, ODSGD_ERR_ARG, "w_bak / grad is NULL");
    if (!c->local[worker_id]) return fail(c, ODSGD_ERR_ARG, "no local buffer for worker " + std::to_string(worker_id));
    const bool need_ms = needs_state(c->local_rule);
    if (need_ms && !c->mean_square[worker_id]) return fail(c, ODSGD_ERR_STATE, "no state arena (mean square / velocity) for that worker");
    const size_t bytes = c->n * sizeof(float);
    StateList st;
    state_buffers(c, &st);
    int rc = check_outside(c, st, Named{grad, "grad", -1});
    if (rc != ODSGD_OK) return rc;
    // the backup may be one of the context's own weight arenas (the replica the pull landed in),
    // but not an arena this call writes
    if (overlap(w_bak, c->local[worker_id], bytes))
        return fail(c, ODSGD_ERR_OVERLAP, "w_bak overlaps local[" + std::to_string(worker_id) + "]");
    if (need_ms && overlap(w_bak, c->mean_square[worker_id], bytes))
        return fail(c, ODSGD_ERR_OVERLAP, "w_bak overlaps mean_square[" + std::to_string(worker_id) + "]");
    LocalArgs a;
    a.w_bak = w_bak;
    a.g = grad;
    a.x = c->local[worker_id];
    a.ms = c->mean_square[worker_id];
    a.w_out = nullptr;
    a.n = c->n;
    a.lp = local_params(c);
    a.lp.first = no_delay ? 1 : 0;
    BufList<4> ptrs;
    ptrs.add(a.w_bak, "w_bak", -1);
    ptrs.add(a.g, "grad", -1);
    ptrs.add(a.x, "local", worker_id);
    if (need_ms) ptrs.add(a.ms, "mean_square", worker_id);
    const int lanes = lanes_for(c, ptrs);
    if (lanes == 0) return ODSGD_ERR_ALIGN;
    rc = before_launch(c, static_cast<cudaStream_t>(stream));
    if (rc != ODSGD_OK) return rc;
    return launch_local(c, a, lanes, false, static_cast<cudaStream_t>(stream));
}

int odsgd_fused_update_host(odsgd_ctx* ctx, const float* const* host_grads, float* const* dev_staging, int worker_id,
                            float* host_local_out, void* stream, void* copy_stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    if (!host_grads || !dev_staging) return fail(c, ODSGD_ERR_ARG, "host_grads / dev_staging is NULL");
    if (worker_id < -1 || worker_id >= c->n_workers) return fail(c, ODSGD_ERR_ARG, "worker_id out of range");
    if (host_local_out && worker_id < 0) return fail(c, ODSGD_ERR_ARG, "host_local_out needs worker_id >= 0");
    for (int m = 0; m < c->n_workers; ++m)
        if (!host_grads[m] || !dev_staging[m]) return fail(c, ODSGD_ERR_ARG, "NULL entry in host_grads / dev_staging");
    // everything that can refuse the update is checked before the first copy is enqueued, so a
    // failed call leaves the staging arenas as they were
    int rc = check_grads(c, dev_staging);
    if (rc != ODSGD_OK) return rc;
    ServerPlan p;
    rc = plan_server(c, dev_staging, true, worker_id, false, nullptr, &p);
    if (rc != ODSGD_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = run_server(c, p, st, true);
    if (rc != ODSGD_OK) return rc;
    cudaStream_t cs = static_cast<cudaStream_t>(copy_stream);
    const bool split = host_local_out && copy_stream && cs != st;
    if (split && (!c->ev_kernel_done || !c->ev_copy_done)) {
        cudaError_t e = cudaSuccess;
        if (!c->ev_kernel_done) e = cudaEventCreateWithFlags(&c->ev_kernel_done, cudaEventDisableTiming);
        if (e == cudaSuccess && !c->ev_copy_done) e = cudaEventCreateWithFlags(&c->ev_copy_done, cudaEventDisableTiming);
        if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("event creation: ") + cudaGetErrorString(e));
    }
    const size_t bytes = c->n * sizeof(float);
    for (int m = 0; m < c->n_workers; ++m) {
        const cudaError_t e = cudaMemcpyAsync(dev_staging[m], host_grads[m], bytes, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("host-to-device copy: ") + cudaGetErrorString(e));
    }
    rc = run_server(c, p, st, false);
    if (rc != ODSGD_OK) return rc;
    if (host_local_out) {
        cudaError_t e = cudaSuccess;
        if (split) {
            e = cudaEventRecord(c->ev_kernel_done, st);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(cs, c->ev_kernel_done, 0);
        }
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(host_local_out, c->local[worker_id], bytes, cudaMemcpyDeviceToHost, split ? cs : st);
        if (e == cudaSuccess && split) {
            e = cudaEventRecord(c->ev_copy_done, cs);
            c->copy_pending = e == cudaSuccess;
            c->copy_waited = false;
        }
        if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("device-to-host copy: ") + cudaGetErrorString(e));
    }
    return ODSGD_OK;
}

int odsgd_asgd_step(odsgd_ctx* ctx, int worker_id, const float* grad, void* stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    if (worker_id < 0 || worker_id >= c->n_workers) return fail(c, ODSGD_ERR_ARG, "worker_id out of range");
    if (!grad) return fail(c, ODSGD_ERR_ARG, "grad is NULL");
    if (!c->v) return fail(c, ODSGD_ERR_STATE, "a worker-only context (ODSGD_FLAG_WORKER_ONLY) has no server state");
    if (c->n_mirrors > 0) return fail(c, ODSGD_ERR_STATE, "weight mirrors are set: the ASGD step would leave them stale");
    StateList st;
    state_buffers(c, &st);
    const int rc_o = check_outside(c, st, Named{grad, "grad", -1});
    if (rc_o != ODSGD_OK) return rc_o;
    AsgdArgs a;
    a.g = grad;
    a.w = c->w[c->cur];
    a.v = c->v;
    a.n = c->n;
    a.lr = c->lr;
    a.momentum = c->momentum;
    a.wd = c->wd;
    BufList<3> ptrs;
    ptrs.add(grad, "grad", -1);
    ptrs.add(a.w, "w", -1);
    ptrs.add(a.v, "v", -1);
    const int lanes = lanes_for(c, ptrs);
    if (lanes == 0) return ODSGD_ERR_ALIGN;
    const int rc_dev = on_own_device(c);
    if (rc_dev != ODSGD_OK) return rc_dev;
    const int rc = launch_asgd(c, a, lanes, static_cast<cudaStream_t>(stream));
    if (rc != ODSGD_OK) return rc;
    c->step += 1;
    c->grads_bound = false;
    c->delayed = nullptr;
    return ODSGD_OK;
}

int odsgd_set_lr(odsgd_ctx* ctx, float lr) {
    if (!ctx) return ODSGD_ERR_ARG;
    ctx->lr = lr;
    return ODSGD_OK;
}

int odsgd_set_local_lr(odsgd_ctx* ctx, float local_lr) {
    if (!ctx) return ODSGD_ERR_ARG;
    ctx->local_lr = local_lr;
    return ODSGD_OK;
}

int odsgd_set_momentum(odsgd_ctx* ctx, float momentum) {
    if (!ctx) return ODSGD_ERR_ARG;
    ctx->momentum = momentum;
    return ODSGD_OK;
}

int odsgd_set_wd(odsgd_ctx* ctx, float wd) {
    if (!ctx) return ODSGD_ERR_ARG;
    ctx->wd = wd;
    return ODSGD_OK;
}

int odsgd_set_local_rule(odsgd_ctx* ctx, int rule, float lambda, float m, float eps, float* const* mean_square) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    if (rule != ODSGD_LOCAL_SGD && rule != ODSGD_LOCAL_DC_C && rule != ODSGD_LOCAL_DC_A && rule != ODSGD_LOCAL_MOMENTUM)
        return fail(c, ODSGD_ERR_ARG, "unknown local rule");
    if (needs_state(rule) && mean_square) {
        const size_t need = (c->flags & ODSGD_FLAG_ALLOW_UNALIGNED) ? 4 : 16;
        for (int w = 0; w < c->n_workers; ++w)
            if (mean_square[w] && !aligned(mean_square[w], need)) return fail(c, ODSGD_ERR_ALIGN, "mean_square arena misaligned");
        float* keep[ODSGD_MAX_WORKERS];
        for (int w = 0; w < c->n_workers; ++w) {
            keep[w] = c->mean_square[w];
            c->mean_square[w] = mean_square[w];
        }
        StateList st;
        state_buffers(c, &st);
        const int rc = check_distinct(c, st, c->n * sizeof(float));
        if (rc != ODSGD_OK) {
            for (int w = 0; w < c->n_workers; ++w) c->mean_square[w] = keep[w];
            return rc;
        }
    } else {
        for (int w = 0; w < c->n_workers; ++w) c->mean_square[w] = nullptr;
    }
    c->state_epoch += 1;  // bound gradient tables were checked against the old set of arenas
    c->local_rule = rule;
    c->dc_lambda = lambda;
    c->dc_m = m;
    c->dc_eps = eps;
    return ODSGD_OK;
}

int odsgd_set_tensor_multipliers(odsgd_ctx* ctx, const float* lr_mult, const float* wd_mult, void* stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    // the table is allocated, filled and freed on the context's own device
    const int rc_dev = on_own_device(c);
    if (rc_dev != ODSGD_OK) return rc_dev;
    // not while `stream` is capturing: the call may allocate, and a captured upload would re-read
    // the context's host copy of the table at every replay (whatever a later call left there)
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(static_cast<cudaStream_t>(stream), &cap) != cudaSuccess) {
        cudaGetLastError();
        return fail(c, ODSGD_ERR_CUDA, "cudaStreamIsCapturing failed");
    }
    if (cap != cudaStreamCaptureStatusNone)
        return fail(c, ODSGD_ERR_STATE, "odsgd_set_tensor_multipliers cannot be recorded into a stream capture");
    if (!lr_mult && !wd_mult) {
        if (c->table_dev) cudaFree(c->table_dev);
        c->table_dev = nullptr;
        c->mult_on = false;
        return ODSGD_OK;
    }
    const size_t nt = c->offsets.size() - 1;
    if (!(c->flags & ODSGD_FLAG_ALLOW_UNALIGNED))
        for (size_t o : c->offsets)
            if (o % 4 != 0)
                return fail(c, ODSGD_ERR_ALIGN, "tensor offset " + std::to_string(o) + " is not a multiple of 4 elements (set ODSGD_FLAG_ALLOW_UNALIGNED for the scalar path)");
    const size_t bytes = (nt + 1) * sizeof(unsigned long long) + 2 * nt * sizeof(float);
    c->table_host.resize(bytes);
    unsigned long long* off = reinterpret_cast<unsigned long long*>(c->table_host.data());
    float* lm = reinterpret_cast<float*>(c->table_host.data() + (nt + 1) * sizeof(unsigned long long));
    float* wm = lm + nt;
    for (size_t t = 0; t <= nt; ++t) off[t] = c->offsets[t];
    for (size_t t = 0; t < nt; ++t) {
        lm[t] = lr_mult ? lr_mult[t] : 1.0f;
        wm[t] = wd_mult ? wd_mult[t] : 1.0f;
    }
    if (!c->table_dev) {
        const cudaError_t e = cudaMalloc(&c->table_dev, bytes);
        if (e != cudaSuccess) {
            c->table_dev = nullptr;
            return fail(c, ODSGD_ERR_CUDA, std::string("multiplier table allocation: ") + cudaGetErrorString(e));
        }
    }
    const cudaError_t e = cudaMemcpyAsync(c->table_dev, c->table_host.data(), bytes, cudaMemcpyHostToDevice,
                                          static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("multiplier table upload: ") + cudaGetErrorString(e));
    c->mult_on = true;
    return ODSGD_OK;
}

int odsgd_set_server_mean_square(odsgd_ctx* ctx, float* mean_square) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    if (mean_square) {
        const size_t need = (c->flags & ODSGD_FLAG_ALLOW_UNALIGNED) ? 4 : 16;
        if (!aligned(mean_square, need)) return fail(c, ODSGD_ERR_ALIGN, "server mean-square arena misaligned");
        float* keep = c->server_ms;
        c->server_ms = nullptr;
        StateList st;
        state_buffers(c, &st);
        const size_t bytes = c->n * sizeof(float);
        for (int i = 0; i < st.n; ++i)
            if (overlap(mean_square, st.b[i].p, bytes)) {
                c->server_ms = keep;
                return fail(c, ODSGD_ERR_OVERLAP, "server mean-square arena overlaps " + label(st.b[i]));
            }
    }
    c->server_ms = mean_square;
    c->state_epoch += 1;
    return ODSGD_OK;
}

int odsgd_set_weight_mirrors(odsgd_ctx* ctx, float* const* mirrors_a, float* const* mirrors_b, int n_mirrors) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    if (n_mirrors < 0 || n_mirrors > ODSGD_MAX_MIRRORS)
        return fail(c, ODSGD_ERR_ARG, "n_mirrors must be in 0.." + std::to_string(ODSGD_MAX_MIRRORS));
    if (n_mirrors == 0) {
        if (c->n_mirrors != 0) c->state_epoch += 1;
        c->n_mirrors = 0;
        return ODSGD_OK;
    }
    if (!c->v) return fail(c, ODSGD_ERR_STATE, "a worker-only context (ODSGD_FLAG_WORKER_ONLY) has no server pass to mirror");
    if (!mirrors_a) return fail(c, ODSGD_ERR_ARG, "mirrors_a is NULL");
    if (c->pingpong && !mirrors_b) return fail(c, ODSGD_ERR_ARG, "the ping-pong layout needs mirrors_b as well");
    if (!c->pingpong && mirrors_b) return fail(c, ODSGD_ERR_ARG, "mirrors_b must be NULL in the in-place layout");
    const size_t need = (c->flags & ODSGD_FLAG_ALLOW_UNALIGNED) ? 4 : 16;
    for (int i = 0; i < n_mirrors; ++i) {
        if (!mirrors_a[i] || (mirrors_b && !mirrors_b[i])) return fail(c, ODSGD_ERR_ARG, "NULL entry in a mirror table");
        if (!aligned(mirrors_a[i], need) || (mirrors_b && !aligned(mirrors_b[i], need)))
            return fail(c, ODSGD_ERR_ALIGN, "mirror " + std::to_string(i) + " is not " + std::to_string(need) + "-byte aligned");
    }
    float* keep[2][ODSGD_MAX_MIRRORS];
    memcpy(keep, c->mirror, sizeof keep);
    const int keep_n = c->n_mirrors;
    for (int i = 0; i < ODSGD_MAX_MIRRORS; ++i) {
        c->mirror[0][i] = i < n_mirrors ? mirrors_a[i] : nullptr;
        c->mirror[1][i] = i < n_mirrors && mirrors_b ? mirrors_b[i] : nullptr;
    }
    c->n_mirrors = n_mirrors;
    StateList st;
    state_buffers(c, &st);
    const int rc = check_distinct(c, st, c->n * sizeof(float));
    if (rc != ODSGD_OK) {
        memcpy(c->mirror, keep, sizeof keep);
        c->n_mirrors = keep_n;
        return rc;
    }
    c->state_epoch += 1;  // bound gradient tables were checked against the old set of buffers
    return ODSGD_OK;
}

int odsgd_dcasgd_step(odsgd_ctx* ctx, int worker_id, const float* grad, void* stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    if (worker_id < 0 || worker_id >= c->n_workers) return fail(c, ODSGD_ERR_ARG, "worker_id out of range");
    if (!grad) return fail(c, ODSGD_ERR_ARG, "grad is NULL");
    if (c->local_rule != ODSGD_LOCAL_DC_C && c->local_rule != ODSGD_LOCAL_DC_A)
        return fail(c, ODSGD_ERR_STATE, "choose ODSGD_LOCAL_DC_C or ODSGD_LOCAL_DC_A with odsgd_set_local_rule first");
    if (!c->local[worker_id]) return fail(c, ODSGD_ERR_ARG, "no backup (local) buffer for worker " + std::to_string(worker_id));
    const bool need_ms = c->local_rule == ODSGD_LOCAL_DC_A;
    if (need_ms && !c->server_ms) return fail(c, ODSGD_ERR_STATE, "ODSGD_LOCAL_DC_A at the server needs odsgd_set_server_mean_square");
    if (c->n_mirrors > 0) return fail(c, ODSGD_ERR_STATE, "weight mirrors are set: the DC-ASGD step would leave them stale");
    StateList st;
    state_buffers(c, &st);
    const int rc_o = check_outside(c, st, Named{grad, "grad", -1});
    if (rc_o != ODSGD_OK) return rc_o;
    LocalArgs a;
    a.w_bak = c->w[c->cur];
    a.w_out = c->w[c->cur];
    a.g = grad;
    a.x = c->local[worker_id];
    a.ms = c->server_ms;
    a.n = c->n;
    a.lp = local_params(c);
    a.lp.local_lr = c->lr;  // the server applies its own learning rate
    BufList<4> ptrs;
    ptrs.add(grad, "grad", -1);
    ptrs.add(a.w_out, "w", -1);
    ptrs.add(a.x, "local", worker_id);
    if (need_ms) ptrs.add(a.ms, "server_mean_square", -1);
    const int lanes = lanes_for(c, ptrs);
    if (lanes == 0) return ODSGD_ERR_ALIGN;
    const int rc_copy = before_launch(c, static_cast<cudaStream_t>(stream));
    if (rc_copy != ODSGD_OK) return rc_copy;
    const int rc = launch_local(c, a, lanes, true, static_cast<cudaStream_t>(stream));
    if (rc != ODSGD_OK) return rc;
    c->step += 1;
    c->grads_bound = false;
    c->delayed = nullptr;
    return ODSGD_OK;
}

int odsgd_set_warmup(odsgd_ctx* ctx, uint64_t wp) {
    if (!ctx) return ODSGD_ERR_ARG;
    if (ctx->iter != 0) return fail(ctx, ODSGD_ERR_STATE, "the warm-up length can only be set before the first odsgd_step");
    ctx->wp = wp;
    return ODSGD_OK;
}

int odsgd_step(odsgd_ctx* ctx, const float* const* worker_grads, void* stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    return scheduled_step(ctx, [&](bool keep_backup, int local_id, bool first) {
        return server_call(ctx, worker_grads, keep_backup, local_id, stream, first);
    });
}

int odsgd_step_bound(odsgd_ctx* ctx, int slot, void* stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    return scheduled_step(ctx, [&](bool keep_backup, int local_id, bool first) {
        return bound_call(ctx, slot, keep_backup, local_id, stream, first);
    });
}

int odsgd_get_train_weights(odsgd_ctx* ctx, int worker_id, float** weights) {
    if (!ctx || !weights) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    if (worker_id < 0 || worker_id >= c->n_workers) return fail(c, ODSGD_ERR_ARG, "worker_id out of range");
    if (c->iter <= c->wp) {
        *weights = c->w[c->cur];
        return ODSGD_OK;
    }
    if (!c->local[worker_id]) return fail(c, ODSGD_ERR_ARG, "no local buffer for worker " + std::to_string(worker_id));
    *weights = c->local[worker_id];
    return ODSGD_OK;
}

int odsgd_get_iteration(odsgd_ctx* ctx, uint64_t* iteration) {
    if (!ctx || !iteration) return ODSGD_ERR_ARG;
    *iteration = ctx->iter;
    return ODSGD_OK;
}

int odsgd_set_iteration(odsgd_ctx* ctx, uint64_t iteration) {
    if (!ctx) return ODSGD_ERR_ARG;
    ctx->iter = iteration;
    return ODSGD_OK;
}

float odsgd_lr_step_decay(float base_lr, float factor, const uint64_t* boundaries, size_t n_boundaries, uint64_t step) {
    double lr = base_lr;
    for (size_t i = 0; i < n_boundaries; ++i)
        if (boundaries && boundaries[i] <= step) lr *= (double)factor;
    return (float)lr;
}

float odsgd_lr_linear_ramp(float start_lr, float end_lr, uint64_t ramp_steps, uint64_t step) {
    if (ramp_steps == 0 || step >= ramp_steps) return end_lr;
    const double f = (double)step / (double)ramp_steps;
    return (float)((double)start_lr + ((double)end_lr - (double)start_lr) * f);
}

float odsgd_lr_poly_decay(float base_lr, float end_lr, float power, uint64_t total_steps, uint64_t step) {
    if (total_steps == 0 || step >= total_steps) return end_lr;
    const double f = 1.0 - (double)step / (double)total_steps;
    return (float)((double)end_lr + ((double)base_lr - (double)end_lr) * pow(f, (double)power));
}

int odsgd_shard_range(size_t n_params, int n_ranks, int rank, size_t* begin, size_t* end) {
    if (!begin || !end || n_ranks < 1 || rank < 0 || rank >= n_ranks) return ODSGD_ERR_ARG;
    // equal slices of ceil(n / R) elements rounded up to 4 (16 bytes); the last ones ragged or empty
    const size_t r = (size_t)n_ranks;
    size_t len = (n_params + r - 1) / r;
    len = (len + 3) / 4 * 4;
    const size_t b = len * (size_t)rank;
    const size_t e = b + len;
    *begin = b < n_params ? b : n_params;
    *end = e < n_params ? e : n_params;
    return ODSGD_OK;
}

int odsgd_get_weights(odsgd_ctx* ctx, float** current, float** delayed) {
    if (!ctx) return ODSGD_ERR_ARG;
    if (current) *current = ctx->w[ctx->cur];
    if (delayed) *delayed = const_cast<float*>(ctx->delayed);
    return ODSGD_OK;
}

int odsgd_get_step(odsgd_ctx* ctx, uint64_t* step) {
    if (!ctx || !step) return ODSGD_ERR_ARG;
    *step = ctx->step;
    return ODSGD_OK;
}

int odsgd_set_step(odsgd_ctx* ctx, uint64_t step) {
    if (!ctx) return ODSGD_ERR_ARG;
    ctx->step = step;
    return ODSGD_OK;
}

int odsgd_set_launch_config(odsgd_ctx* ctx, int block_threads, int ctas_per_sm) {
    if (!ctx) return ODSGD_ERR_ARG;
    if (block_threads != 0 && (block_threads < 64 || block_threads > 1024 || block_threads % 32 != 0))
        return fail(ctx, ODSGD_ERR_ARG, "block_threads must be 0 or a multiple of 32 in 64..1024");
    if (ctas_per_sm < 0) return fail(ctx, ODSGD_ERR_ARG, "ctas_per_sm must be >= 0");
    ctx->block_threads = block_threads;
    ctx->ctas_per_sm = ctas_per_sm;
    return ODSGD_OK;
}

int odsgd_get_launch_count(odsgd_ctx* ctx, uint64_t* launches) {
    if (!ctx || !launches) return ODSGD_ERR_ARG;
    *launches = ctx->launches;
    return ODSGD_OK;
}

// ---------------------------------------------------------------------------------------
// Allocation-free variant of the fused update with per-tensor multipliers.
//
// Callers that may not cudaMalloc (a server loop that cannot take cudaMalloc's device-wide
// synchronisation; a process whose device memory belongs to a framework pool) get the
// multiplier table from g_static_table, a fixed array in the library image, instead of the
// table odsgd_set_tensor_multipliers() allocates.  The name g_static_table is a device
// symbol: host code must not pass it to a kernel as if it were an address.  Its device
// address is looked up once per device with cudaGetSymbolAddress (static_table_address) and
// that pointer is what the kernel receives.
}  // extern "C"

static __device__ __align__(256) unsigned char g_static_table[ODSGD_STATIC_TABLE_BYTES];

namespace {

constexpr int kMaxDevices = 64;
unsigned char* g_static_table_addr[kMaxDevices] = {};  // per device: address of g_static_table there
unsigned char g_static_stage[ODSGD_STATIC_TABLE_BYTES];  // host copy the upload reads from (no allocation)
// One lock for the address cache and the host staging array: both are shared by every
// context, device and thread of the process.
std::mutex g_static_mutex;

// Device address of g_static_table on the current device; looked up on first use.
// Call with g_static_mutex held.
int static_table_address(odsgd_ctx* c, unsigned char** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return fail(c, ODSGD_ERR_UNSUPPORTED, "device ordinal beyond the static table's bookkeeping");
    if (dev != c->device) return fail(c, ODSGD_ERR_STATE, "the context was created on another device than the current one");
    if (!g_static_table_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_table);
        if (e != cudaSuccess || !p) {
            cudaGetLastError();
            return fail(c, ODSGD_ERR_CUDA, std::string("cudaGetSymbolAddress(static table): ") + cudaGetErrorString(e));
        }
        g_static_table_addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_static_table_addr[dev];
    return ODSGD_OK;
}

}  // namespace

extern "C" {

int odsgd_fused_update_mult_static(odsgd_ctx* ctx, const float* const* worker_grads, int worker_id,
                                   const float* lr_mult, const float* wd_mult, void* stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
    if (worker_id < 0 || worker_id >= c->n_workers) return fail(c, ODSGD_ERR_ARG, "worker_id out of range");
    if (!c->local[worker_id]) return fail(c, ODSGD_ERR_ARG, "no local buffer for worker " + std::to_string(worker_id));
    if (c->local_rule != ODSGD_LOCAL_SGD)
        return fail(c, ODSGD_ERR_UNSUPPORTED, "the allocation-free call supports the ODSGD_LOCAL_SGD rule only");
    const size_t nt = c->offsets.size() - 1;
    if (nt > ODSGD_STATIC_MAX_TENSORS)
        return fail(c, ODSGD_ERR_UNSUPPORTED, std::to_string(nt) + " tensors exceed the static table's limit of " +
                                                  std::to_string(ODSGD_STATIC_MAX_TENSORS) +
                                                  " (use odsgd_set_tensor_multipliers + odsgd_fused_update)");
    if (!c->offsets_vec_ok && !(c->flags & ODSGD_FLAG_ALLOW_UNALIGNED))
        return fail(c, ODSGD_ERR_ALIGN, "a tensor offset is not a multiple of 4 elements (set ODSGD_FLAG_ALLOW_UNALIGNED for the scalar path)");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Under stream capture the table upload would become a graph node that re-reads the shared
    // host staging array at every replay, i.e. whatever table the last eager call of any context
    // left there: refuse instead.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) {
        cudaGetLastError();
        return fail(c, ODSGD_ERR_CUDA, "cudaStreamIsCapturing failed");
    }
    if (cap != cudaStreamCaptureStatusNone)
        return fail(c, ODSGD_ERR_STATE, "odsgd_fused_update_mult_static cannot be recorded into a stream capture");

    int rc = check_grads(c, worker_grads);
    if (rc != ODSGD_OK) return rc;

    // From here to the return of the upload the shared host staging array is in use: one call
    // at a time in the whole process, whatever the device.
    std::lock_guard<std::mutex> lock(g_static_mutex);
    unsigned char* table = nullptr;
    rc = static_table_address(c, &table);
    if (rc != ODSGD_OK) return rc;
    ServerPlan p;
    rc = plan_server(c, worker_grads, true, worker_id, false, table, &p);
    if (rc != ODSGD_OK) return rc;
    rc = run_server(c, p, st, true);
    if (rc != ODSGD_OK) return rc;

    // table layout: offsets u64 x (T+1) | lr_mult f32 x T | wd_mult f32 x T; every entry the
    // kernel will read is rewritten here, so nothing depends on what an earlier call left
    const size_t bytes = (nt + 1) * sizeof(unsigned long long) + 2 * nt * sizeof(float);
    unsigned long long* off = reinterpret_cast<unsigned long long*>(g_static_stage);
    float* lm = reinterpret_cast<float*>(g_static_stage + (nt + 1) * sizeof(unsigned long long));
    float* wm = lm + nt;
    for (size_t t = 0; t <= nt; ++t) off[t] = c->offsets[t];
    for (size_t t = 0; t < nt; ++t) {
        lm[t] = lr_mult ? lr_mult[t] : 1.0f;
        wm[t] = wd_mult ? wd_mult[t] : 1.0f;
    }
    // the source is pageable host memory: when this returns, the runtime has taken its own copy
    // of the bytes, so the staging array may be refilled by the next caller
    const cudaError_t e = cudaMemcpyAsync(table, g_static_stage, bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("static table upload: ") + cudaGetErrorString(e));
    return run_server(c, p, st, false);
}

const char* odsgd_last_error(odsgd_ctx* ctx) {
    return ctx ? ctx->err.c_str() : g_create_err.c_str();
}

}  // extern "C"
