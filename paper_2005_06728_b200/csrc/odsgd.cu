// Host side of the OD-SGD update library: context, validation, kernel selection
// and launches behind the C ABI declared in odsgd.h.  No torch types, no
// allocation of parameter-sized memory, no synchronisation.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
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
    float* v = nullptr;
    float* local[ODSGD_MAX_WORKERS] = {};
    float* mean_square[ODSGD_MAX_WORKERS] = {};
    size_t n = 0;
    std::vector<size_t> offsets;
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
    uint64_t wp = 0;             // Algorithm 2's warm-up length
    uint64_t iter = 0;           // iterations done through odsgd_step
    // host-buffer entry point with a separate copy stream: ordering between the two streams
    cudaEvent_t ev_kernel_done = nullptr;  // recorded on the compute stream after the update kernel
    cudaEvent_t ev_copy_done = nullptr;    // recorded on the copy stream after the device-to-host copy
    bool copy_pending = false;
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

// State buffers of a context, for alias checks.
std::vector<Named> state_buffers(const odsgd_ctx* c) {
    std::vector<Named> s;
    s.push_back({c->w[0], "w_a", -1});
    if (c->w[1]) s.push_back({c->w[1], "w_b", -1});
    if (c->w_delayed) s.push_back({c->w_delayed, "w_delayed", -1});
    s.push_back({c->v, "v", -1});
    for (int m = 0; m < c->n_workers; ++m) {
        if (c->local[m]) s.push_back({c->local[m], "local", m});
        if (c->mean_square[m]) s.push_back({c->mean_square[m], "mean_square", m});
    }
    if (c->server_ms) s.push_back({c->server_ms, "server_mean_square", -1});
    return s;
}

int check_distinct(odsgd_ctx* err_ctx, const std::vector<Named>& s, size_t bytes) {
    for (size_t i = 0; i < s.size(); ++i)
        for (size_t j = i + 1; j < s.size(); ++j)
            if (overlap(s[i].p, s[j].p, bytes))
                return fail(err_ctx, ODSGD_ERR_OVERLAP, label(s[i]) + " overlaps " + label(s[j]));
    return ODSGD_OK;
}

// Vector width usable for a call: 4 lanes when every pointer is 16-byte aligned, else
// 1 lane if the context allows it.  Returns 0 and sets the error otherwise.
int lanes_for(odsgd_ctx* c, const std::vector<Named>& ptrs) {
    bool all16 = true;
    for (const Named& b : ptrs) {
        if (!aligned(b.p, 4)) {
            fail(c, ODSGD_ERR_ALIGN, label(b) + " is not 4-byte aligned");
            return 0;
        }
        if (!aligned(b.p, 16)) {
            if (!(c->flags & ODSGD_FLAG_ALLOW_UNALIGNED)) {
                fail(c, ODSGD_ERR_ALIGN, label(b) + " is not 16-byte aligned (set ODSGD_FLAG_ALLOW_UNALIGNED for the scalar path)");
                return 0;
            }
            all16 = false;
        }
    }
    return all16 ? 4 : 1;
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

int too_wide(odsgd_ctx* c, int block) {
    return fail(c, ODSGD_ERR_UNSUPPORTED, "block_threads = " + std::to_string(block) + " is too large for this kernel");
}

template <bool DET, int NL, int LOCAL, int RULE, bool MULT, int BB, int UB>
int launch_server_k(odsgd_ctx* c, const ServerArgs& a, cudaStream_t st) {
    const int block = c->block_threads > 0 ? c->block_threads : kDefaultBlock;
    auto kernel = server_kernel<DET, NL, LOCAL, RULE, MULT, BB, UB>;
    if (resident_cached(c, kernel, block) == 0) return too_wide(c, block);
    const int grid = grid_for(c, a.n, NL, block, UB, kServerCtasPerSm);
    kernel<<<grid, block, 0, st>>>(a);
    return after_launch(c, "server kernel launch");
}

template <bool DET, int NL, int LOCAL, int RULE, bool MULT>
int launch_server_m(odsgd_ctx* c, const ServerArgs& a, cudaStream_t st) {
    // few workers: the pass is close to a copy and wants the shallow, wide shape
    if constexpr (LOCAL != kLocalAll) {
        if (a.n_workers <= kFewWorkers)
            return launch_server_k<DET, NL, LOCAL, RULE, MULT, kFewBatch, kFewUnroll>(c, a, st);
    }
    return launch_server_k<DET, NL, LOCAL, RULE, MULT, kBatch, kUnroll>(c, a, st);
}

template <bool DET, int NL, int LOCAL, int RULE>
int launch_server_t(odsgd_ctx* c, const ServerArgs& a, cudaStream_t st) {
    return c->mult_on ? launch_server_m<DET, NL, LOCAL, RULE, true>(c, a, st)
                      : launch_server_m<DET, NL, LOCAL, RULE, false>(c, a, st);
}

template <bool DET, int NL, int LOCAL>
int launch_server_r(odsgd_ctx* c, const ServerArgs& a, cudaStream_t st) {
    if (LOCAL == kLocalNone) return launch_server_t<DET, NL, LOCAL, ODSGD_LOCAL_SGD>(c, a, st);
    switch (c->local_rule) {
        case ODSGD_LOCAL_SGD: return launch_server_t<DET, NL, LOCAL, ODSGD_LOCAL_SGD>(c, a, st);
        case ODSGD_LOCAL_DC_C: return launch_server_t<DET, NL, LOCAL, ODSGD_LOCAL_DC_C>(c, a, st);
        case ODSGD_LOCAL_MOMENTUM: return launch_server_t<DET, NL, LOCAL, ODSGD_LOCAL_MOMENTUM>(c, a, st);
        default: return launch_server_t<DET, NL, LOCAL, ODSGD_LOCAL_DC_A>(c, a, st);
    }
}

template <bool DET, int NL>
int launch_server_l(odsgd_ctx* c, const ServerArgs& a, int local_mode, cudaStream_t st) {
    switch (local_mode) {
        case kLocalNone: return launch_server_r<DET, NL, kLocalNone>(c, a, st);
        case kLocalOne: return launch_server_r<DET, NL, kLocalOne>(c, a, st);
        default: return launch_server_r<DET, NL, kLocalAll>(c, a, st);
    }
}

int launch_server(odsgd_ctx* c, const ServerArgs& a, int lanes, int local_mode, cudaStream_t st) {
    const bool det = (c->flags & ODSGD_FLAG_ALLOW_FMA) == 0;
    if (det) return lanes == 4 ? launch_server_l<true, 4>(c, a, local_mode, st) : launch_server_l<true, 1>(c, a, local_mode, st);
    return lanes == 4 ? launch_server_l<false, 4>(c, a, local_mode, st) : launch_server_l<false, 1>(c, a, local_mode, st);
}

template <bool DET, int NL, int RULE, bool SERVER>
int launch_local_t(odsgd_ctx* c, const LocalArgs& a, cudaStream_t st) {
    const int block = c->block_threads > 0 ? c->block_threads : kDefaultSmallBlock;
    auto kernel = local_kernel<DET, NL, RULE, SERVER>;
    if (resident_cached(c, kernel, block) == 0) return too_wide(c, block);
    kernel<<<grid_for(c, a.n, NL, block, kSmallUnroll, kServerCtasPerSm), block, 0, st>>>(a);
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
    const int block = c->block_threads > 0 ? c->block_threads : kDefaultSmallBlock;
    auto kernel = asgd_kernel<DET, NL>;
    if (resident_cached(c, kernel, block) == 0) return too_wide(c, block);
    kernel<<<grid_for(c, a.n, NL, block, kSmallUnroll, kServerCtasPerSm), block, 0, st>>>(a);
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

// Run before every kernel launch: the context's device must be current, and a copy-back of
// local weights that odsgd_fused_update_host put on a separate copy stream must be out before
// a later kernel overwrites a local arena (`st` is made to wait for it).
int before_launch(odsgd_ctx* c, cudaStream_t st) {
    const int rc_dev = on_own_device(c);
    if (rc_dev != ODSGD_OK) return rc_dev;
    if (!c->copy_pending) return ODSGD_OK;
    const cudaError_t e = cudaStreamWaitEvent(st, c->ev_copy_done, 0);
    if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("stream wait: ") + cudaGetErrorString(e));
    c->copy_pending = false;
    return ODSGD_OK;
}

// Checks a table of gradient pointers against the context's state buffers.
int check_grads(odsgd_ctx* c, const float* const* grads, std::vector<Named>* ptrs) {
    if (!grads) return fail(c, ODSGD_ERR_ARG, "worker_grads is NULL");
    const size_t bytes = c->n * sizeof(float);
    const std::vector<Named> st = state_buffers(c);
    for (int m = 0; m < c->n_workers; ++m) {
        if (!grads[m]) return fail(c, ODSGD_ERR_ARG, "worker_grads[" + std::to_string(m) + "] is NULL");
        const Named g{grads[m], "worker_grads", m};
        for (const Named& s : st)
            if (overlap(g.p, s.p, bytes)) return fail(c, ODSGD_ERR_OVERLAP, label(g) + " overlaps " + label(s));
        ptrs->push_back(g);
    }
    return ODSGD_OK;
}

// Local mode and outputs for a fused call; fills a.x / a.ms / a.local_worker.
int bind_local_outputs(odsgd_ctx* c, int worker_id, ServerArgs* a, int* local_mode, std::vector<Named>* ptrs) {
    if (worker_id >= c->n_workers || worker_id < -1) return fail(c, ODSGD_ERR_ARG, "worker_id out of range");
    const bool need_ms = needs_state(c->local_rule);
    if (worker_id >= 0) {
        if (!c->local[worker_id]) return fail(c, ODSGD_ERR_ARG, "no local buffer for worker " + std::to_string(worker_id));
        if (need_ms && !c->mean_square[worker_id]) return fail(c, ODSGD_ERR_STATE, "no mean-square arena for that worker");
        a->x[0] = c->local[worker_id];
        a->ms[0] = c->mean_square[worker_id];
        a->local_worker = worker_id;
        ptrs->push_back({a->x[0], "local", worker_id});
        if (need_ms) ptrs->push_back({a->ms[0], "mean_square", worker_id});
        *local_mode = kLocalOne;
        return ODSGD_OK;
    }
    int count = 0;
    for (int m = 0; m < c->n_workers; ++m) {
        a->x[m] = c->local[m];
        a->ms[m] = c->mean_square[m];
        if (c->local[m]) {
            if (need_ms && !c->mean_square[m]) return fail(c, ODSGD_ERR_STATE, "no mean-square arena for worker " + std::to_string(m));
            ptrs->push_back({a->x[m], "local", m});
            if (need_ms) ptrs->push_back({a->ms[m], "mean_square", m});
            ++count;
        }
    }
    if (count == 0) return fail(c, ODSGD_ERR_ARG, "worker_id == -1 but the context has no local buffers");
    *local_mode = kLocalAll;
    return ODSGD_OK;
}

// Shared body of the global, fused and SSGD calls.
//   keep_backup: OD-SGD server step (the old weights stay available to the workers)
//   local_id:    -2 none, -1 all workers, >= 0 one worker
int server_call(odsgd_ctx* c, const float* const* grads, bool keep_backup, int local_id, void* stream,
                bool first_delayed_step = false) {
    if (!c) return ODSGD_ERR_ARG;
    std::vector<Named> ptrs;
    int rc = check_grads(c, grads, &ptrs);
    if (rc != ODSGD_OK) return rc;

    ServerArgs a;
    memset(&a, 0, sizeof a);
    for (int m = 0; m < c->n_workers; ++m) a.g[m] = grads[m];
    a.v = c->v;
    a.n = c->n;
    a.n_workers = c->n_workers;
    a.inv_n = 1.0f / (float)c->n_workers;
    a.lr = c->lr;
    a.momentum = c->momentum;
    a.wd = c->wd;
    a.lp = local_params(c);
    a.lp.first = first_delayed_step ? 1 : 0;
    if (c->mult_on) {
        const size_t nt = c->offsets.size() - 1;
        unsigned char* base = static_cast<unsigned char*>(c->table_dev);
        a.t_off = reinterpret_cast<const unsigned long long*>(base);
        a.t_lr_mult = reinterpret_cast<const float*>(base + (nt + 1) * sizeof(unsigned long long));
        a.t_wd_mult = a.t_lr_mult + nt;
        a.n_tensors = (unsigned int)nt;
    }
    a.w_in = c->w[c->cur];
    const float* delayed_after = nullptr;
    int next_cur = c->cur;
    if (keep_backup && c->pingpong) {
        a.w_out = c->w[c->cur ^ 1];
        delayed_after = c->w[c->cur];
        next_cur = c->cur ^ 1;
    } else {
        a.w_out = c->w[c->cur];
        if (keep_backup && c->w_delayed) {
            a.w_prev = c->w_delayed;
            delayed_after = c->w_delayed;
        }
    }
    ptrs.push_back({a.w_in, "w", -1});
    ptrs.push_back({a.w_out, "w", -1});
    ptrs.push_back({a.v, "v", -1});
    if (a.w_prev) ptrs.push_back({a.w_prev, "w_delayed", -1});

    int local_mode = kLocalNone;
    if (local_id >= -1) {
        rc = bind_local_outputs(c, local_id, &a, &local_mode, &ptrs);
        if (rc != ODSGD_OK) return rc;
    }
    int lanes = lanes_for(c, ptrs);
    if (lanes == 0) return ODSGD_ERR_ALIGN;
    if (c->mult_on && lanes == 4) {
        // a 128-bit vector must not straddle two tensors (set_tensor_multipliers has checked that
        // the scalar path is allowed when it would)
        for (size_t o : c->offsets)
            if (o % 4 != 0) { lanes = 1; break; }
    }

    rc = before_launch(c, static_cast<cudaStream_t>(stream));
    if (rc != ODSGD_OK) return rc;
    rc = launch_server(c, a, lanes, local_mode, static_cast<cudaStream_t>(stream));
    if (rc != ODSGD_OK) return rc;

    c->cur = next_cur;
    c->step += 1;
    c->delayed = delayed_after;
    c->grads_bound = keep_backup;
    if (keep_backup)
        for (int m = 0; m < c->n_workers; ++m) c->bound[m] = grads[m];
    return ODSGD_OK;
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
    if (!d->w_a || !d->v) return fail(nullptr, ODSGD_ERR_ARG, "w_a and v must not be NULL");
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
    if (d->flags & ~(ODSGD_FLAG_DETERMINISTIC | ODSGD_FLAG_ALLOW_UNALIGNED | ODSGD_FLAG_ALLOW_FMA))
        return fail(nullptr, ODSGD_ERR_ARG, "unknown flag bits");
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
    c->lr = d->lr;
    c->local_lr = d->local_lr;
    c->momentum = d->momentum;
    c->wd = d->wd;
    c->flags = d->flags;
    if (d->local)
        for (int m = 0; m < d->n_workers; ++m) c->local[m] = d->local[m];

    const std::vector<Named> st = state_buffers(c);
    const size_t need = (d->flags & ODSGD_FLAG_ALLOW_UNALIGNED) ? 4 : 16;
    for (const Named& b : st) {
        if (!aligned(b.p, need)) {
            const std::string msg = label(b) + " is not " + std::to_string(need) + "-byte aligned";
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
    std::vector<Named> ptrs = {{a.w_bak, "w_delayed", -1}, {a.g, "worker_grads", worker_id}, {a.x, "local", worker_id}};
    if (need_ms) ptrs.push_back({a.ms, "mean_square", worker_id});
    const int lanes = lanes_for(c, ptrs);
    if (lanes == 0) return ODSGD_ERR_ALIGN;
    const int rc_copy = before_launch(c, static_cast<cudaStream_t>(stream));
    if (rc_copy != ODSGD_OK) return rc_copy;
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
    // validate before the first copy is enqueued
    std::vector<Named> ptrs;
    int rc = check_grads(c, dev_staging, &ptrs);
    if (rc != ODSGD_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t bytes = c->n * sizeof(float);
    for (int m = 0; m < c->n_workers; ++m) {
        const cudaError_t e = cudaMemcpyAsync(dev_staging[m], host_grads[m], bytes, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("host-to-device copy: ") + cudaGetErrorString(e));
    }
    cudaStream_t cs = static_cast<cudaStream_t>(copy_stream);
    const bool split = host_local_out && copy_stream && cs != st;
    if (split && (!c->ev_kernel_done || !c->ev_copy_done)) {
        cudaError_t e = cudaSuccess;
        if (!c->ev_kernel_done) e = cudaEventCreateWithFlags(&c->ev_kernel_done, cudaEventDisableTiming);
        if (e == cudaSuccess && !c->ev_copy_done) e = cudaEventCreateWithFlags(&c->ev_copy_done, cudaEventDisableTiming);
        if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("event creation: ") + cudaGetErrorString(e));
    }
    rc = server_call(c, dev_staging, true, worker_id, stream);
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
    const size_t bytes = c->n * sizeof(float);
    const Named g{grad, "grad", -1};
    for (const Named& s : state_buffers(c))
        if (overlap(g.p, s.p, bytes)) return fail(c, ODSGD_ERR_OVERLAP, "grad overlaps " + label(s));
    AsgdArgs a;
    a.g = grad;
    a.w = c->w[c->cur];
    a.v = c->v;
    a.n = c->n;
    a.lr = c->lr;
    a.momentum = c->momentum;
    a.wd = c->wd;
    const int lanes = lanes_for(c, {g, {a.w, "w", -1}, {a.v, "v", -1}});
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
        odsgd_ctx probe = *c;
        for (int w = 0; w < c->n_workers; ++w) probe.mean_square[w] = mean_square[w];
        const std::vector<Named> st = state_buffers(&probe);
        const size_t need = (c->flags & ODSGD_FLAG_ALLOW_UNALIGNED) ? 4 : 16;
        for (int w = 0; w < c->n_workers; ++w)
            if (mean_square[w] && !aligned(mean_square[w], need)) return fail(c, ODSGD_ERR_ALIGN, "mean_square arena misaligned");
        const int rc = check_distinct(c, st, c->n * sizeof(float));
        if (rc != ODSGD_OK) return rc;
        for (int w = 0; w < c->n_workers; ++w) c->mean_square[w] = mean_square[w];
    } else {
        for (int w = 0; w < c->n_workers; ++w) c->mean_square[w] = nullptr;
    }
    c->local_rule = rule;
    c->dc_lambda = lambda;
    c->dc_m = m;
    c->dc_eps = eps;
    return ODSGD_OK;
}

int odsgd_set_tensor_multipliers(odsgd_ctx* ctx, const float* lr_mult, const float* wd_mult, void* stream) {
    if (!ctx) return ODSGD_ERR_ARG;
    odsgd_ctx* c = ctx;
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
        const size_t bytes = c->n * sizeof(float);
        float* keep = c->server_ms;
        c->server_ms = nullptr;
        for (const Named& s : state_buffers(c))
            if (overlap(mean_square, s.p, bytes)) {
                c->server_ms = keep;
                return fail(c, ODSGD_ERR_OVERLAP, "server mean-square arena overlaps " + label(s));
            }
    }
    c->server_ms = mean_square;
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
    const size_t bytes = c->n * sizeof(float);
    const Named g{grad, "grad", -1};
    for (const Named& s : state_buffers(c))
        if (overlap(g.p, s.p, bytes)) return fail(c, ODSGD_ERR_OVERLAP, "grad overlaps " + label(s));
    LocalArgs a;
    a.w_bak = c->w[c->cur];
    a.w_out = c->w[c->cur];
    a.g = grad;
    a.x = c->local[worker_id];
    a.ms = c->server_ms;
    a.n = c->n;
    a.lp = local_params(c);
    a.lp.local_lr = c->lr;  // the server applies its own learning rate
    std::vector<Named> ptrs = {g, {a.w_out, "w", -1}, {a.x, "local", worker_id}};
    if (need_ms) ptrs.push_back({a.ms, "server_mean_square", -1});
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
    odsgd_ctx* c = ctx;
    int rc;
    if (c->iter < c->wp) {
        rc = server_call(c, worker_grads, false, -2, stream);  // warm-up stage: SSGD
    } else {
        // from the last warm-up iteration on: server step + local update of every worker; at
        // iteration wp itself the gradients were taken on the global weights (no delay yet)
        rc = server_call(c, worker_grads, true, -1, stream, c->iter == c->wp);
    }
    if (rc == ODSGD_OK) c->iter += 1;
    return rc;
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

// Device address of g_static_table on the current device; looked up on first use.
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
    bool vec_ok = true;
    for (size_t o : c->offsets)
        if (o % 4 != 0) vec_ok = false;
    if (!vec_ok && !(c->flags & ODSGD_FLAG_ALLOW_UNALIGNED))
        return fail(c, ODSGD_ERR_ALIGN, "a tensor offset is not a multiple of 4 elements (set ODSGD_FLAG_ALLOW_UNALIGNED for the scalar path)");

    std::vector<Named> ptrs;
    int rc = check_grads(c, worker_grads, &ptrs);
    if (rc != ODSGD_OK) return rc;
    unsigned char* table = nullptr;
    rc = static_table_address(c, &table);
    if (rc != ODSGD_OK) return rc;

    ServerArgs a;
    memset(&a, 0, sizeof a);
    for (int m = 0; m < c->n_workers; ++m) a.g[m] = worker_grads[m];
    a.v = c->v;
    a.n = c->n;
    a.n_workers = c->n_workers;
    a.inv_n = 1.0f / (float)c->n_workers;
    a.lr = c->lr;
    a.momentum = c->momentum;
    a.wd = c->wd;
    a.lp = local_params(c);
    a.w_in = c->w[c->cur];
    const float* delayed_after = nullptr;
    int next_cur = c->cur;
    if (c->pingpong) {
        a.w_out = c->w[c->cur ^ 1];
        delayed_after = c->w[c->cur];
        next_cur = c->cur ^ 1;
    } else {
        a.w_out = c->w[c->cur];
        if (c->w_delayed) {
            a.w_prev = c->w_delayed;
            delayed_after = c->w_delayed;
        }
    }
    a.x[0] = c->local[worker_id];
    a.local_worker = worker_id;
    ptrs.push_back({a.w_in, "w", -1});
    ptrs.push_back({a.w_out, "w", -1});
    ptrs.push_back({a.v, "v", -1});
    ptrs.push_back({a.x[0], "local", worker_id});
    if (a.w_prev) ptrs.push_back({a.w_prev, "w_delayed", -1});
    int lanes = lanes_for(c, ptrs);
    if (lanes == 0) return ODSGD_ERR_ALIGN;
    if (!vec_ok) lanes = 1;

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
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const cudaError_t e = cudaMemcpyAsync(table, g_static_stage, bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return fail(c, ODSGD_ERR_CUDA, std::string("static table upload: ") + cudaGetErrorString(e));
    a.t_off = reinterpret_cast<const unsigned long long*>(table);
    a.t_lr_mult = reinterpret_cast<const float*>(table + (nt + 1) * sizeof(unsigned long long));
    a.t_wd_mult = a.t_lr_mult + nt;
    a.n_tensors = (unsigned int)nt;

    rc = before_launch(c, st);
    if (rc != ODSGD_OK) return rc;
    const bool det = (c->flags & ODSGD_FLAG_ALLOW_FMA) == 0;
    if (det)
        rc = lanes == 4 ? launch_server_m<true, 4, kLocalOne, ODSGD_LOCAL_SGD, true>(c, a, st)
                        : launch_server_m<true, 1, kLocalOne, ODSGD_LOCAL_SGD, true>(c, a, st);
    else
        rc = lanes == 4 ? launch_server_m<false, 4, kLocalOne, ODSGD_LOCAL_SGD, true>(c, a, st)
                        : launch_server_m<false, 1, kLocalOne, ODSGD_LOCAL_SGD, true>(c, a, st);
    if (rc != ODSGD_OK) return rc;
    c->cur = next_cur;
    c->step += 1;
    c->delayed = delayed_after;
    c->grads_bound = true;
    for (int m = 0; m < c->n_workers; ++m) c->bound[m] = worker_grads[m];
    return ODSGD_OK;
}

const char* odsgd_last_error(odsgd_ctx* ctx) {
    return ctx ? ctx->err.c_str() : g_create_err.c_str();
}

}  // extern "C"
