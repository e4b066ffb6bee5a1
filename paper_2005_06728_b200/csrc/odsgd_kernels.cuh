// Device code of the OD-SGD update pass for sm_100a.
//
// All rules are element-wise and bound by HBM bandwidth (about a quarter of a
// flop per byte), so the kernels are organised around memory traffic only:
//   * every input stream is read exactly once and every output written once;
//   * 128-bit loads and stores, each warp touching 512 contiguous bytes per
//     stream per instruction, each CTA walking contiguous tiles of every stream;
//   * the M gradient streams are fetched in batches of B x U independent
//     128-bit loads per thread (B workers x U vectors) before the dependent adds
//     start: 8 x 2 with many workers (about 160 KB in flight per SM at two
//     resident CTAs), shapes with a batch that divides the worker count and more
//     vectors per thread when there are few (server_shape_for); the adds
//     themselves stay in worker order 0..M-1; with every worker's local update
//     fused in, shallower batches win (each worker's result leaves at once);
//   * gradients go through the read-only path (ld.global.nc), which measured
//     5-8 % faster here than streaming loads (ld.global.cs); state that is read
//     and written by the same kernel uses coherent loads; results are stored
//     with the streaming policy;
//   * one launch covers the whole arena whatever the number of tensors in it: a
//     grid capped per SM (server_grid_cap) strides over the tiles, close to one
//     tile per CTA when tiles are heavy so that the hardware scheduler evens out
//     the tail, close to persistent for the copy-like one-worker pass;
//   * every kernel opens with the two programmatic-dependent-launch instructions: it lets the
//     next kernel of the stream be scheduled at once (griddepcontrol.launch_dependents) and
//     itself waits, before its first memory access, until the kernels ahead of it have
//     completed and their writes are visible (griddepcontrol.wait).  Launched with the
//     matching attribute, back-to-back update kernels no longer pay the full launch latency
//     between them, which is most of an iteration on the small, cache-resident parameter sets;
//     launched without it, both instructions do nothing.
// Tensor cores have no role here: there is no contraction.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "odsgd.h"

namespace odsgd {

// ------------------------------------------------------------------ tuning constants
// Each can be overridden with -D for a sweep; the defaults are what measured best on B200.

// Server kernel, many workers: gradient loads per batch x vectors per thread.
#ifndef ODSGD_BATCH
#define ODSGD_BATCH 8
#endif
#ifndef ODSGD_UNROLL
#define ODSGD_UNROLL 2
#endif
// Server kernel with every worker's local update in the pass.  Each worker's result is stored as
// soon as its gradient is in, so few workers per round of loads and more vectors per thread do
// best: plain rule 2 x 4 (against 8 x 2: +2 % at M = 32, +4 % at M = 4, +13 % at M = 2 on the
// 138 M-parameter arena, equal on the others; 3 x 4 and 2 x 5 tie, 1 x 4, 1 x 6, 2 x 6 lose 3-8 %);
// Eq. 4: one worker per round, 2 vectors, 128-thread CTAs (+2 % over 1 vector x 256 threads; 3
// vectors lose 4 %); Eq. 5-6 and local momentum: one worker, one vector, 128-thread CTAs (+2 %
// for Eq. 5-6; two or four workers per round change it by less than 1 %, two vectors cost 3-4 %).
#ifndef ODSGD_ALLSGD_BATCH
#define ODSGD_ALLSGD_BATCH 2
#endif
#ifndef ODSGD_ALLSGD_UNROLL
#define ODSGD_ALLSGD_UNROLL 4
#endif
#ifndef ODSGD_ALLDC_BATCH
#define ODSGD_ALLDC_BATCH 1
#endif
#ifndef ODSGD_ALLDC_UNROLL
#define ODSGD_ALLDC_UNROLL 1
#endif
#ifndef ODSGD_ALLDCC_UNROLL
#define ODSGD_ALLDCC_UNROLL 2
#endif
// Block size of the all-workers variants with a delay-compensated or momentum local rule.
#ifndef ODSGD_ALLDC_BLOCK
#define ODSGD_ALLDC_BLOCK 128
#endif
// One worker's delay-compensated or momentum local update in the pass: where its extra arenas
// are read and where it is computed.
//   ODSGD_ONE_INLINE    the update is computed and stored the moment that worker's gradient comes
//                       by in the sum, its extra arenas fetched with the weights at the top of
//                       the tile, instead of after the server rule behind one more dependent
//                       round of loads: 0 never, 1 for the rules with a state arena, 2 for Eq. 4
//                       as well, 3 for every rule.  Measured against 0 (fused update, one worker):
//                       Eq. 4 +8 % at M = 8, +16 % at M = 4, +2 % at M = 16; Eq. 5-6 +6 %, +9 %,
//                       +3.5 % (although 16-48 bytes spill); local momentum +7.5 %, +13 %, +3 %;
//                       the plain rule within +-0.5 % (it has no extra arena to wait for).
//   ODSGD_ONE_DC_EARLY  only where the update is not inline: Eq. 4's previous local weights are
//                       fetched at the top of the tile but used after the server rule: 0 never,
//                       1 with two vectors per thread or fewer, 2 always (ties with inline, 0.4 %
//                       ahead at M = 16, but spills up to 192 bytes in the 3 x 4 shape).
// Issuing worker m + 1's loads ahead of worker m's stores in the all-workers variants (a software
// pipeline over the workers) was measured too and lost 1-3 %.
#ifndef ODSGD_ONE_DC_EARLY
#define ODSGD_ONE_DC_EARLY 1
#endif
#ifndef ODSGD_ONE_INLINE
#define ODSGD_ONE_INLINE 2
#endif
// ASGD kernel / local kernel: vectors per thread per tile.  The local kernel with the plain rule
// (two streams in, one out) does 1 % better with three than with four on all three large arenas,
// the ASGD kernel 0.2-0.6 % better with four; two or six lose 0.5-1 % in both.
#ifndef ODSGD_SMALL_UNROLL
#define ODSGD_SMALL_UNROLL 4
#endif
#ifndef ODSGD_LOCAL_UNROLL
#define ODSGD_LOCAL_UNROLL 3
#endif
// Gradient loads: 0 streaming (ld.global.cs), 1 read-only path (ld.global.nc), 2 default caching,
// 3 read-only path without L1 allocation and a 256-byte L2 prefetch hint, 4 read-only path without
// L1 allocation under an L2 evict-first policy.
#ifndef ODSGD_GRAD_LOAD
#define ODSGD_GRAD_LOAD 1
#endif
// Stores: 0 streaming (st.global.cs), 1 default caching, 2 under an L2 evict-first policy.
#ifndef ODSGD_STORE
#define ODSGD_STORE 0
#endif
// Register cap of the server kernel: __launch_bounds__(ODSGD_MAX_BLOCK, ODSGD_MIN_CTAS).  512 x 1
// allows 128 registers per thread, i.e. two resident CTAs of the default 256 threads; without
// the cap the Eq. 5-6 instantiations take 131-141 registers and lose the second CTA (measured:
// 4.6 instead of 6.9 TB/s).  Launches wider than ODSGD_MAX_BLOCK threads are refused by the host.
#ifndef ODSGD_MIN_CTAS
#define ODSGD_MIN_CTAS 1
#endif
#ifndef ODSGD_MAX_BLOCK
#define ODSGD_MAX_BLOCK 512
#endif

constexpr int kBatch = ODSGD_BATCH;
constexpr int kUnroll = ODSGD_UNROLL;
constexpr int kAllSgdBatch = ODSGD_ALLSGD_BATCH;
constexpr int kAllSgdUnroll = ODSGD_ALLSGD_UNROLL;
constexpr int kAllDcBatch = ODSGD_ALLDC_BATCH;
constexpr int kAllDcUnroll = ODSGD_ALLDC_UNROLL;
constexpr int kAllDcCUnroll = ODSGD_ALLDCC_UNROLL;
constexpr int kSmallUnroll = ODSGD_SMALL_UNROLL;
constexpr int kLocalUnroll = ODSGD_LOCAL_UNROLL;
constexpr int kOneDcEarly = ODSGD_ONE_DC_EARLY;
constexpr int kOneInline = ODSGD_ONE_INLINE;
#if ODSGD_MIN_CTAS > 0
#define ODSGD_SERVER_BOUNDS __launch_bounds__(ODSGD_MAX_BLOCK, ODSGD_MIN_CTAS)
#else
#define ODSGD_SERVER_BOUNDS
#endif

// Launch shape (used by the host side; kept here so that everything that decides how the
// kernels touch memory lives in one file).
constexpr int kDefaultBlock = 256;       // server kernel
constexpr int kDefaultLocalBlock = 512;  // local kernel
constexpr int kDefaultAsgdBlock = 256;   // ASGD kernel (256 against 512 threads: +0.6-1.4 % on the mid-size arenas)
// Grid cap in CTAs per SM; the grid strides over the tiles beyond it.  How much a CTA should
// loop depends on how heavy a tile is.  With many gradient streams a tile is hundreds of KB and
// finer-grained scheduling evens out the tail: 256 per SM (in effect one tile per CTA) measured
// 0.6-1.9 % faster than 64 from M = 4 up, and than an exactly persistent grid.  The copy-like
// one-worker pass has light tiles and sits in between: 32 per SM (against 16: +1 % on the 61 M-
// and 138 M-parameter arenas, equal on the 25 M one; 64 gains another 1 % on the large two and
// loses 2.4 % on the small one); two workers take 64.
constexpr int kLocalCtasPerSm = 128;
constexpr int kAsgdCtasPerSm = 256;
__host__ __device__ constexpr int server_grid_cap(int n_workers) {
    return n_workers <= 1 ? 32 : (n_workers == 2 ? 64 : 256);
}

// What else the server pass carries: nothing, one worker's local update, every worker's, or -
// with no local update - a copy of the new weights into each of the context's weight mirrors
// (the other ranks' replicas when the server role is sharded: the pull of Section 2.2 done by
// the kernel's own stores instead of a collective behind it).
enum LocalMode : int { kLocalNone = 0, kLocalOne = 1, kLocalAll = 2, kLocalNoneMirrored = 3 };

// Launch shape of the server kernel by worker count M: gradient loads per batch x vectors per
// thread.  A batch that M divides evenly leaves no half-empty round of loads, and the fewer the
// streams, the more vectors per thread it takes to keep enough bytes in flight.  Measured on
// the 138 M-parameter arena (GB/s of algorithmic bytes, fused update), best shape per M:
//   M <= 2: 2 x 4        M = 3, 5, 6, 9: 3 x 4        M = 4, 7, 8, 10..12: 4 x 3        M > 12: 8 x 2
// (3 x 4 against 8 x 2: +3 % at M = 3, +4 % at M = 5 and 9; 4 x 3 against 8 x 2: +2 % at M = 12;
// 8 x 2 against 4 x 3 at M = 13..16: +0-1 % with the plain local rule, +1-3 % with a
// delay-compensated one, whose early fetch of the previous local weights needs two vectors or
// fewer; 4 x 4, 6 x 3, 2 x 5 and 2 x 6 spill registers or lose 15-25 %.)
enum ServerShape : int { kShape2x4 = 0, kShape3x4 = 1, kShape4x3 = 2, kShapeMany = 3 };
// The three few-worker shapes as batch x vectors (overridable for a sweep, like the rest).
#ifndef ODSGD_SHAPE0_B
#define ODSGD_SHAPE0_B 2
#endif
#ifndef ODSGD_SHAPE0_U
#define ODSGD_SHAPE0_U 4
#endif
#ifndef ODSGD_SHAPE1_B
#define ODSGD_SHAPE1_B 3
#endif
#ifndef ODSGD_SHAPE1_U
#define ODSGD_SHAPE1_U 4
#endif
#ifndef ODSGD_SHAPE2_B
#define ODSGD_SHAPE2_B 4
#endif
#ifndef ODSGD_SHAPE2_U
#define ODSGD_SHAPE2_U 3
#endif
__host__ __device__ constexpr int server_shape_for(int n_workers) {
    return n_workers <= 2 ? kShape2x4
           : (n_workers == 3 || n_workers == 5 || n_workers == 6 || n_workers == 9) ? kShape3x4
           : n_workers <= 12 ? kShape4x3
                             : kShapeMany;
}

// Vectors per thread per tile of the server kernel: UB as instantiated, except when the pass
// also carries every worker's local update (fewer when that update is delay-compensated and
// touches three arenas per worker: registers are the scarce resource there).  The kernel and
// the host-side grid sizing both take the tile from here.
__host__ __device__ constexpr int server_vectors_per_thread(int local_mode, int rule, int ub) {
    return local_mode != kLocalAll      ? ub
           : rule == ODSGD_LOCAL_SGD    ? kAllSgdUnroll
           : rule == ODSGD_LOCAL_DC_C   ? kAllDcCUnroll
                                        : kAllDcUnroll;
}

// Threads per CTA the host launches by default.  The local kernel's Eq. 5-6 instantiation (four
// streams in, two out, a square root and a division per element) does 4-5 % better in 256-thread
// CTAs than in 512-thread ones; the other rules are within 1 % either way.
__host__ __device__ constexpr int local_default_block(int rule) {
    return rule == ODSGD_LOCAL_DC_A ? 256 : kDefaultLocalBlock;
}
__host__ __device__ constexpr int server_default_block(int local_mode, int rule) {
    return local_mode == kLocalAll && rule != ODSGD_LOCAL_SGD ? ODSGD_ALLDC_BLOCK : kDefaultBlock;
}

struct LocalParams {
    float local_lr;
    float lambda;       // Eq. 4 / Eq. 5 compensation coefficient
    float m;            // Eq. 6 decay
    float one_minus_m;  // computed once on the host in fp32
    float eps;          // Eq. 5
    int first;          // 1: the gradient was computed on w_bak itself (first delayed step), x_prev := w_bak
};

// Kernel argument block, passed by value (constant bank): no dependent device
// load is needed to find a worker's gradient buffer.
struct ServerArgs {
    const float* g[ODSGD_MAX_WORKERS];  // gradient arenas, worker order
    float* x[ODSGD_MAX_WORKERS];        // local-weight arenas (kLocalAll) or x[0] (kLocalOne)
    float* ms[ODSGD_MAX_WORKERS];       // Eq. 6 state, same indexing as x
    const float* w_in;                  // weights before the update
    float* w_out;                       // weights after the update (may equal w_in)
    float* w_prev;                      // optional copy of the old weights
    float* v;                           // momentum state, in place
    float* w_mirror[ODSGD_MAX_MIRRORS]; // kLocalNoneMirrored: further destinations of the new weights
    int n_mirrors;
    unsigned long long n;               // elements
    int n_workers;
    int local_worker;                   // kLocalOne: whose gradient feeds x[0]
    float inv_n;                        // 1.0f / n_workers, computed on the host
    float lr, momentum, wd;
    LocalParams lp;
    // per-tensor multipliers (MULT kernels only): device table, n_tensors + 1 ascending offsets
    const unsigned long long* t_off;
    const float* t_lr_mult;
    const float* t_wd_mult;
    unsigned int n_tensors;
};

struct LocalArgs {
    const float* w_bak;
    const float* g;
    float* x;      // read (previous local weights) by the delay-compensated rules, then written
    float* ms;     // Eq. 6 state or null
    float* w_out;  // server-side DC-ASGD only: the global weights, which receive the result too
    unsigned long long n;
    LocalParams lp;
};

struct AsgdArgs {
    const float* g;
    float* w;
    float* v;
    unsigned long long n;
    float lr, momentum, wd;
};

// ------------------------------------------------------------------ dependent launch
// 1: launch with programmatic stream serialization (0 keeps the instructions, drops the attribute).
#ifndef ODSGD_PDL
#define ODSGD_PDL 1
#endif
constexpr bool kProgrammaticLaunch = ODSGD_PDL != 0;

__device__ __forceinline__ void dependent_launch_prologue() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ------------------------------------------------------------------ vectors
template <int NL>
struct Vec {
    float e[NL];
};

template <int NL>
__device__ __forceinline__ Vec<NL> load_stream(const float* p);
template <>
__device__ __forceinline__ Vec<4> load_stream<4>(const float* p) {
    const float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    return Vec<4>{{t.x, t.y, t.z, t.w}};
}
template <>
__device__ __forceinline__ Vec<1> load_stream<1>(const float* p) {
    return Vec<1>{{__ldcs(p)}};
}

// Gradients (and the backup weights of the local kernel) are never written by the kernel
// that reads them, so they may also go through the read-only path.
template <int NL>
__device__ __forceinline__ Vec<NL> load_grad(const float* p);
#if ODSGD_GRAD_LOAD == 4 || ODSGD_STORE == 2
__device__ __forceinline__ unsigned long long evict_first_policy() {
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
#endif

template <>
__device__ __forceinline__ Vec<4> load_grad<4>(const float* p) {
#if ODSGD_GRAD_LOAD == 1
    const float4 t = __ldg(reinterpret_cast<const float4*>(p));
#elif ODSGD_GRAD_LOAD == 2
    const float4 t = *reinterpret_cast<const float4*>(p);
#elif ODSGD_GRAD_LOAD == 3
    float4 t;
    asm volatile("ld.global.nc.L1::no_allocate.L2::256B.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(t.x), "=f"(t.y), "=f"(t.z), "=f"(t.w) : "l"(p));
#elif ODSGD_GRAD_LOAD == 4
    float4 t;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(t.x), "=f"(t.y), "=f"(t.z), "=f"(t.w) : "l"(p), "l"(evict_first_policy()));
#else
    const float4 t = __ldcs(reinterpret_cast<const float4*>(p));
#endif
    return Vec<4>{{t.x, t.y, t.z, t.w}};
}
template <>
__device__ __forceinline__ Vec<1> load_grad<1>(const float* p) {
#if ODSGD_GRAD_LOAD == 1
    return Vec<1>{{__ldg(p)}};
#elif ODSGD_GRAD_LOAD == 2
    return Vec<1>{{*p}};
#else
    return Vec<1>{{__ldcs(p)}};
#endif
}

template <int NL>
__device__ __forceinline__ void store_stream(float* p, const Vec<NL>& a);
template <>
__device__ __forceinline__ void store_stream<4>(float* p, const Vec<4>& a) {
#if ODSGD_STORE == 1
    *reinterpret_cast<float4*>(p) = make_float4(a.e[0], a.e[1], a.e[2], a.e[3]);
#elif ODSGD_STORE == 2
    asm volatile("st.global.L1::no_allocate.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;"
                 :: "l"(p), "f"(a.e[0]), "f"(a.e[1]), "f"(a.e[2]), "f"(a.e[3]), "l"(evict_first_policy()) : "memory");
#else
    __stcs(reinterpret_cast<float4*>(p), make_float4(a.e[0], a.e[1], a.e[2], a.e[3]));
#endif
}
template <>
__device__ __forceinline__ void store_stream<1>(float* p, const Vec<1>& a) {
#if ODSGD_STORE == 1
    *p = a.e[0];
#else
    __stcs(p, a.e[0]);
#endif
}

// ------------------------------------------------------------------ arithmetic
// DET: each operator is its own correctly rounded binary32 operation (the
// intrinsics are never contracted).  Otherwise plain operators, which the
// compiler may contract into fused multiply-adds.
template <bool DET>
struct Op {
    static __device__ __forceinline__ float add(float a, float b) { return DET ? __fadd_rn(a, b) : a + b; }
    static __device__ __forceinline__ float sub(float a, float b) { return DET ? __fsub_rn(a, b) : a - b; }
    static __device__ __forceinline__ float mul(float a, float b) { return DET ? __fmul_rn(a, b) : a * b; }
    static __device__ __forceinline__ float div(float a, float b) { return DET ? __fdiv_rn(a, b) : a / b; }
    static __device__ __forceinline__ float sqrt(float a) { return DET ? __fsqrt_rn(a) : sqrtf(a); }
};

// Momentum SGD with L2 decay on one element (Algorithm 1's "Update w_t").
template <bool DET>
__device__ __forceinline__ void server_rule(float gbar, float w, float v, float lr, float momentum, float wd,
                                            float& w_new, float& v_new) {
    using O = Op<DET>;
    const float d = O::add(gbar, O::mul(wd, w));
    v_new = O::sub(O::mul(momentum, v), O::mul(lr, d));
    w_new = O::add(w, v_new);
}

// Local updater on one element (Section 3.3).  x_prev / ms are only touched by
// the delay-compensated rules.
// Which extra arenas a local rule touches: the worker's previous local weights (Eq. 4, Eq. 5)
// and a per-worker state arena (Eq. 6's mean square, or the velocity of local momentum SGD).
__host__ __device__ constexpr bool needs_prev(int rule) { return rule == ODSGD_LOCAL_DC_C || rule == ODSGD_LOCAL_DC_A; }
__host__ __device__ constexpr bool needs_state(int rule) { return rule == ODSGD_LOCAL_DC_A || rule == ODSGD_LOCAL_MOMENTUM; }

template <bool DET, int RULE>
__device__ __forceinline__ float local_rule(float w_bak, float g, float x_prev, float& ms, const LocalParams& p) {
    using O = Op<DET>;
    if (RULE == ODSGD_LOCAL_SGD) {
        return O::sub(w_bak, O::mul(p.local_lr, g));
    }
    if (RULE == ODSGD_LOCAL_MOMENTUM) {
        // the server's rule run by the worker: state = velocity, m = local momentum, lambda = local decay
        float x, u;
        server_rule<DET>(g, w_bak, ms, p.local_lr, p.m, p.lambda, x, u);
        ms = u;
        return x;
    }
    const float gg = O::mul(g, g);
    float lam = p.lambda;
    if (RULE == ODSGD_LOCAL_DC_A) {
        ms = O::add(O::mul(p.m, ms), O::mul(p.one_minus_m, gg));  // Eq. 6
        lam = O::div(p.lambda, O::sqrt(O::add(ms, p.eps)));
    }
    const float diff = O::sub(w_bak, x_prev);
    const float comp = O::mul(O::mul(lam, gg), diff);
    return O::sub(w_bak, O::mul(p.local_lr, O::add(g, comp)));  // Eq. 4 / Eq. 5
}

// ------------------------------------------------------------------ per-tensor multipliers
// Which tensor an element belongs to: binary search over the offset table (a few hundred
// entries at most, L1/L2 resident), skipped while the thread stays inside the tensor it
// found last (the large tensors hold almost all elements).
struct TensorCursor {
    unsigned long long lo = 1, hi = 0;  // empty range: the first lookup searches
    float lr_mult = 1.0f, wd_mult = 1.0f;
};

__device__ __forceinline__ void find_tensor(const ServerArgs& a, unsigned long long off, TensorCursor& c) {
    if (off >= c.lo && off < c.hi) return;
    unsigned int lo = 0, hi = a.n_tensors;  // t_off[lo] <= off < t_off[hi]
    while (hi - lo > 1) {
        const unsigned int mid = (lo + hi) >> 1;
        if (__ldg(a.t_off + mid) <= off) lo = mid; else hi = mid;
    }
    c.lo = __ldg(a.t_off + lo);
    c.hi = __ldg(a.t_off + lo + 1);
    c.lr_mult = __ldg(a.t_lr_mult + lo);
    c.wd_mult = __ldg(a.t_wd_mult + lo);
}

// ------------------------------------------------------------------ server kernel
// One vector (NL lanes) of the arena at element offset `off`:
// sum the workers in order, apply the server rule, and (LOCAL != none) the
// local rule for one worker or for every worker that has a local buffer.
template <bool DET, int NL, int LOCAL, int RULE, bool MULT, int BB, int U>
__device__ __forceinline__ void server_vectors(const ServerArgs& a, const unsigned long long (&off)[U],
                                               const bool (&ok)[U], TensorCursor& cur) {
    using O = Op<DET>;
    Vec<NL> w[U], v[U], s[U], gl[U];
    // one worker's local update with extra arenas: inline in the sum, or fetched early (see
    // ODSGD_ONE_INLINE / ODSGD_ONE_DC_EARLY)
    constexpr bool kInline = LOCAL == kLocalOne &&
                             (kOneInline == 3 || (kOneInline == 2 && RULE != ODSGD_LOCAL_SGD) ||
                              (kOneInline == 1 && needs_state(RULE)));
    constexpr bool kOneDc = LOCAL == kLocalOne && (needs_prev(RULE) || needs_state(RULE)) &&
                            (kInline || (!needs_state(RULE) && kOneDcEarly == 1 && U <= 2) ||
                             (!needs_state(RULE) && kOneDcEarly == 2));
    Vec<NL> xe[kOneDc ? U : 1], mse[kOneDc ? U : 1];
    // Where a worker's previous local weights are read from.  On the first delayed step the
    // gradient was taken on w_bak itself, so x_prev := w_bak: the same loads, pointed at the
    // weights.  (A pointer select, not a conditional load: with the choice made per load, the
    // loads of a tile were no longer issued together, which cost the one-worker Eq. 4 / Eq. 5-6
    // passes 3-16 % and the local kernel 16-42 %.)  Every element's x_prev is read before the
    // same thread stores that element of w_out, so the in-place layout reads the old weights.
    const float* xprev_one = a.lp.first ? a.w_in : a.x[0];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (ok[u]) {
            w[u] = load_stream<NL>(a.w_in + off[u]);
            v[u] = load_stream<NL>(a.v + off[u]);
            if (kOneDc) {
                if (needs_prev(RULE)) xe[u] = load_stream<NL>(xprev_one + off[u]);
                if (needs_state(RULE)) mse[u] = load_stream<NL>(a.ms[0] + off[u]);
            }
        }
    }
    // With every worker's delay-compensated local update in the pass, the previous local weights
    // (and mean squares) are fetched in the same batch as the gradients, so a smaller batch
    // keeps the register count in check.
    constexpr bool kAllDc = LOCAL == kLocalAll && RULE != ODSGD_LOCAL_SGD;
    constexpr int B = kAllDc ? kAllDcBatch : (LOCAL == kLocalAll ? kAllSgdBatch : BB);
    const int n_workers = a.n_workers;
    for (int m0 = 0; m0 < n_workers; m0 += B) {
        Vec<NL> t[B][U], xv[B][U], msv[B][U];
        // independent loads first ...
#pragma unroll
        for (int j = 0; j < B; ++j) {
            if (m0 + j < n_workers) {
                const float* gp = a.g[m0 + j];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (ok[u]) t[j][u] = load_grad<NL>(gp + off[u]);
                }
                if (kAllDc) {
                    float* xp = a.x[m0 + j];
                    if (xp != nullptr) {
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            if (ok[u]) {
                                if (needs_prev(RULE)) xv[j][u] = load_stream<NL>((a.lp.first ? a.w_in : xp) + off[u]);
                                if (needs_state(RULE)) msv[j][u] = load_stream<NL>(a.ms[m0 + j] + off[u]);
                            }
                        }
                    }
                }
            }
        }
        // ... then the adds, strictly in worker order
#pragma unroll
        for (int j = 0; j < B; ++j) {
            const int m = m0 + j;
            if (m < n_workers) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (ok[u]) {
                        if (m == 0) {
                            s[u] = t[j][u];
                        } else {
#pragma unroll
                            for (int l = 0; l < NL; ++l) s[u].e[l] = O::add(s[u].e[l], t[j][u].e[l]);
                        }
                        if (LOCAL == kLocalOne) {
                            if (m == a.local_worker) {
                                if (kInline) {
                                    Vec<NL> xo;
#pragma unroll
                                    for (int l = 0; l < NL; ++l) {
                                        xo.e[l] = local_rule<DET, RULE>(w[u].e[l], t[j][u].e[l], xe[kOneDc ? u : 0].e[l],
                                                                        mse[kOneDc ? u : 0].e[l], a.lp);
                                    }
                                    store_stream<NL>(a.x[0] + off[u], xo);
                                    if (needs_state(RULE)) store_stream<NL>(a.ms[0] + off[u], mse[kOneDc ? u : 0]);
                                } else {
                                    gl[u] = t[j][u];
                                }
                            }
                        }
                        if (LOCAL == kLocalAll) {
                            float* xp = a.x[m];
                            if (xp != nullptr) {
                                Vec<NL> xo;
#pragma unroll
                                for (int l = 0; l < NL; ++l) {
                                    xo.e[l] = local_rule<DET, RULE>(w[u].e[l], t[j][u].e[l], xv[j][u].e[l],
                                                                    msv[j][u].e[l], a.lp);
                                }
                                store_stream<NL>(xp + off[u], xo);
                                if (needs_state(RULE)) store_stream<NL>(a.ms[m] + off[u], msv[j][u]);
                            }
                        }
                    }
                }
            }
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (!ok[u]) continue;
        Vec<NL> wn, vn;
        float lr = a.lr, wd = a.wd;
        if (MULT) {  // lr_t = lr * lr_mult[t], wd_t = wd * wd_mult[t], one rounding each
            find_tensor(a, off[u], cur);
            lr = O::mul(a.lr, cur.lr_mult);
            wd = O::mul(a.wd, cur.wd_mult);
        }
#pragma unroll
        for (int l = 0; l < NL; ++l) {
            const float gbar = O::mul(s[u].e[l], a.inv_n);
            server_rule<DET>(gbar, w[u].e[l], v[u].e[l], lr, a.momentum, wd, wn.e[l], vn.e[l]);
        }
        if (LOCAL == kLocalOne && !kInline) {
            float* xp = a.x[0];
            Vec<NL> xo, xv, msv;
            if (kOneDc) {
                xv = xe[u];
                msv = mse[u];
            } else {
                if (needs_prev(RULE)) xv = load_stream<NL>(xprev_one + off[u]);
                if (needs_state(RULE)) msv = load_stream<NL>(a.ms[0] + off[u]);
            }
#pragma unroll
            for (int l = 0; l < NL; ++l) {
                xo.e[l] = local_rule<DET, RULE>(w[u].e[l], gl[u].e[l], xv.e[l], msv.e[l], a.lp);
            }
            store_stream<NL>(xp + off[u], xo);
            if (needs_state(RULE)) store_stream<NL>(a.ms[0] + off[u], msv);
        }
        if (a.w_prev != nullptr) store_stream<NL>(a.w_prev + off[u], w[u]);
        store_stream<NL>(a.v + off[u], vn);
        store_stream<NL>(a.w_out + off[u], wn);
        if (LOCAL == kLocalNoneMirrored) {
            // the same vector to every mirror (plain stores: a mirror may be peer-mapped memory
            // of another GPU, reached over NVLink)
            for (int r = 0; r < a.n_mirrors; ++r) store_stream<NL>(a.w_mirror[r] + off[u], wn);
        }
    }
}

// BB x UB: gradient loads per batch x vectors per thread (server_shape_for picks them).
template <bool DET, int NL, int LOCAL, int RULE, bool MULT, int BB, int UB>
__global__ void ODSGD_SERVER_BOUNDS server_kernel(const __grid_constant__ ServerArgs a) {
    dependent_launch_prologue();
    TensorCursor cur;
    constexpr int UU = server_vectors_per_thread(LOCAL, RULE, UB);
    const unsigned long long nvec = a.n / NL;
    const unsigned long long tile = (unsigned long long)blockDim.x * UU;
    const unsigned long long stride = (unsigned long long)gridDim.x * tile;
    for (unsigned long long base = (unsigned long long)blockIdx.x * tile; base < nvec; base += stride) {
        unsigned long long off[UU];
        bool ok[UU];
#pragma unroll
        for (int u = 0; u < UU; ++u) {
            const unsigned long long i = base + (unsigned long long)u * blockDim.x + threadIdx.x;
            ok[u] = i < nvec;
            off[u] = i * NL;
        }
        server_vectors<DET, NL, LOCAL, RULE, MULT, BB, UU>(a, off, ok, cur);
    }
    if (NL > 1) {
        // ragged tail: the last n % NL elements, one lane each
        const unsigned long long done = nvec * NL;
        if (blockIdx.x == 0 && done + threadIdx.x < a.n) {
            const unsigned long long off1[1] = {done + threadIdx.x};
            const bool ok1[1] = {true};
            server_vectors<DET, 1, LOCAL, RULE, MULT, BB, 1>(a, off1, ok1, cur);
        }
    }
}

// ------------------------------------------------------------------ local kernel
// Few streams per element (2-4 reads, 1-2 writes): each thread takes kLocalUnroll vectors per
// tile and issues all their loads before the first store, which is what a plain copy needs
// to approach the copy ceiling of the part.
// SERVER = true is DC-ASGD at the parameter server (Eq. 4 / Eq. 5 applied to an arriving
// gradient): w_bak is then the live global vector, read coherently and overwritten with the
// result, and x is the worker's backup copy, which receives the same result (the worker pulls).
template <bool DET, int NL, int RULE, bool SERVER, int U>
__device__ __forceinline__ void local_vectors(const LocalArgs& a, const unsigned long long (&off)[U],
                                              const bool (&ok)[U]) {
    Vec<NL> w[U], g[U], xv[U], msv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (ok[u]) {
            w[u] = SERVER ? load_stream<NL>(a.w_bak + off[u]) : load_grad<NL>(a.w_bak + off[u]);
            g[u] = load_grad<NL>(a.g + off[u]);
            if (needs_prev(RULE)) xv[u] = load_stream<NL>((a.lp.first ? a.w_bak : a.x) + off[u]);
            if (needs_state(RULE)) msv[u] = load_stream<NL>(a.ms + off[u]);
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (!ok[u]) continue;
        Vec<NL> xo;
#pragma unroll
        for (int l = 0; l < NL; ++l) xo.e[l] = local_rule<DET, RULE>(w[u].e[l], g[u].e[l], xv[u].e[l], msv[u].e[l], a.lp);
        store_stream<NL>(a.x + off[u], xo);
        if (SERVER) store_stream<NL>(a.w_out + off[u], xo);
        if (needs_state(RULE)) store_stream<NL>(a.ms + off[u], msv[u]);
    }
}

template <bool DET, int NL, int RULE, bool SERVER>
__global__ void local_kernel(const __grid_constant__ LocalArgs a) {
    dependent_launch_prologue();
    const unsigned long long nvec = a.n / NL;
    const unsigned long long tile = (unsigned long long)blockDim.x * kLocalUnroll;
    const unsigned long long stride = (unsigned long long)gridDim.x * tile;
    for (unsigned long long base = (unsigned long long)blockIdx.x * tile; base < nvec; base += stride) {
        unsigned long long off[kLocalUnroll];
        bool ok[kLocalUnroll];
#pragma unroll
        for (int u = 0; u < kLocalUnroll; ++u) {
            const unsigned long long i = base + (unsigned long long)u * blockDim.x + threadIdx.x;
            ok[u] = i < nvec;
            off[u] = i * NL;
        }
        local_vectors<DET, NL, RULE, SERVER, kLocalUnroll>(a, off, ok);
    }
    if (NL > 1) {
        const unsigned long long done = nvec * NL;
        if (blockIdx.x == 0 && done + threadIdx.x < a.n) {
            const unsigned long long off1[1] = {done + threadIdx.x};
            const bool ok1[1] = {true};
            local_vectors<DET, 1, RULE, SERVER, 1>(a, off1, ok1);
        }
    }
}

// ------------------------------------------------------------------ ASGD kernel
template <bool DET, int NL, int U>
__device__ __forceinline__ void asgd_vectors(const AsgdArgs& a, const unsigned long long (&off)[U], const bool (&ok)[U]) {
    Vec<NL> g[U], w[U], v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (ok[u]) {
            g[u] = load_grad<NL>(a.g + off[u]);
            w[u] = load_stream<NL>(a.w + off[u]);
            v[u] = load_stream<NL>(a.v + off[u]);
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        if (!ok[u]) continue;
        Vec<NL> wn, vn;
#pragma unroll
        for (int l = 0; l < NL; ++l)
            server_rule<DET>(g[u].e[l], w[u].e[l], v[u].e[l], a.lr, a.momentum, a.wd, wn.e[l], vn.e[l]);
        store_stream<NL>(a.v + off[u], vn);
        store_stream<NL>(a.w + off[u], wn);
    }
}

template <bool DET, int NL>
__global__ void asgd_kernel(const __grid_constant__ AsgdArgs a) {
    dependent_launch_prologue();
    const unsigned long long nvec = a.n / NL;
    const unsigned long long tile = (unsigned long long)blockDim.x * kSmallUnroll;
    const unsigned long long stride = (unsigned long long)gridDim.x * tile;
    for (unsigned long long base = (unsigned long long)blockIdx.x * tile; base < nvec; base += stride) {
        unsigned long long off[kSmallUnroll];
        bool ok[kSmallUnroll];
#pragma unroll
        for (int u = 0; u < kSmallUnroll; ++u) {
            const unsigned long long i = base + (unsigned long long)u * blockDim.x + threadIdx.x;
            ok[u] = i < nvec;
            off[u] = i * NL;
        }
        asgd_vectors<DET, NL, kSmallUnroll>(a, off, ok);
    }
    if (NL > 1) {
        const unsigned long long done = nvec * NL;
        if (blockIdx.x == 0 && done + threadIdx.x < a.n) {
            const unsigned long long off1[1] = {done + threadIdx.x};
            const bool ok1[1] = {true};
            asgd_vectors<DET, 1, 1>(a, off1, ok1);
        }
    }
}

}  // namespace odsgd
