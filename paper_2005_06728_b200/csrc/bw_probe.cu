// Memory-bandwidth ceilings of the GPU the update kernels run on, measured with the same
// access styles the kernels could use: pure reads with 128-bit read-only loads, with 256-bit
// loads, and with TMA bulk copies (cp.async.bulk) into a shared-memory ring; and 1:1 copies.
// The update kernels are judged against these: a read-dominated kernel can sit between the
// copy figure and the pure-read figure, never above the latter.
//
// Every spin on an mbarrier is bounded; if one gives up, the kernel raises a flag, waits
// (bounded) for its copies in flight and returns.
// Standalone program: built by paper_2005_06728_b200/bw_probe.py, prints one line per case.
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdlib>
#include <cstdint>
#include <vector>

#define CK(x) do { cudaError_t e = (x); if (e != cudaSuccess) { printf("CUDA error %s at %s:%d\n", cudaGetErrorString(e), __FILE__, __LINE__); exit(1);} } while (0)

// ---------------------------------------------------------------- 128-bit read, K streams, U vectors/thread
template <int K, int U>
__global__ void read128(const float4* __restrict__ base, size_t stream_vecs, size_t nvec, float* sink) {
    float acc = 0.f;
    const size_t tile = (size_t)blockDim.x * U;
    for (size_t b = (size_t)blockIdx.x * tile; b < nvec; b += (size_t)gridDim.x * tile) {
        float4 t[K][U];
#pragma unroll
        for (int k = 0; k < K; ++k)
#pragma unroll
            for (int u = 0; u < U; ++u) {
                size_t i = b + (size_t)u * blockDim.x + threadIdx.x;
                if (i < nvec) t[k][u] = __ldg(base + (size_t)k * stream_vecs + i); else t[k][u] = make_float4(0, 0, 0, 0);
            }
#pragma unroll
        for (int k = 0; k < K; ++k)
#pragma unroll
            for (int u = 0; u < U; ++u) acc += t[k][u].x + t[k][u].y + t[k][u].z + t[k][u].w;
    }
    if (acc == 1234.5678f) sink[threadIdx.x] = acc;
}

// ---------------------------------------------------------------- 256-bit read
struct alignas(32) F8 { float v[8]; };
__device__ __forceinline__ F8 ld256(const F8* p) {
    F8 r;
    asm volatile("ld.global.nc.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
                 : "l"(p));
    return r;
}
template <int K, int U>
__global__ void read256(const F8* __restrict__ base, size_t stream_vecs, size_t nvec, float* sink) {
    float acc = 0.f;
    const size_t tile = (size_t)blockDim.x * U;
    for (size_t b = (size_t)blockIdx.x * tile; b < nvec; b += (size_t)gridDim.x * tile) {
        F8 t[K][U];
#pragma unroll
        for (int k = 0; k < K; ++k)
#pragma unroll
            for (int u = 0; u < U; ++u) {
                size_t i = b + (size_t)u * blockDim.x + threadIdx.x;
                if (i < nvec) t[k][u] = ld256(base + (size_t)k * stream_vecs + i);
                else { for (int q = 0; q < 8; ++q) t[k][u].v[q] = 0.f; }
            }
#pragma unroll
        for (int k = 0; k < K; ++k)
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int q = 0; q < 8; ++q) acc += t[k][u].v[q];
    }
    if (acc == 1234.5678f) sink[threadIdx.x] = acc;
}

// ---------------------------------------------------------------- copy 128-bit
template <int U>
__global__ void copy128(const float4* __restrict__ src, float4* __restrict__ dst, size_t nvec) {
    const size_t tile = (size_t)blockDim.x * U;
    for (size_t b = (size_t)blockIdx.x * tile; b < nvec; b += (size_t)gridDim.x * tile) {
        float4 t[U];
#pragma unroll
        for (int u = 0; u < U; ++u) { size_t i = b + (size_t)u * blockDim.x + threadIdx.x; if (i < nvec) t[u] = __ldg(src + i); }
#pragma unroll
        for (int u = 0; u < U; ++u) { size_t i = b + (size_t)u * blockDim.x + threadIdx.x; if (i < nvec) __stcs(dst + i, t[u]); }
    }
}

// ---------------------------------------------------------------- TMA bulk read into a smem ring
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// TILE bytes per stage, S stages; tiles are distributed round-robin over CTAs.
template <int TILE, int S>
__global__ void read_tma(const char* __restrict__ base, size_t n_tiles, float* sink, int* err) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t full[S];
    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int s = 0; s < S; ++s) mbar_init(&full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const size_t first = blockIdx.x, step = gridDim.x;
    size_t my_tiles = first < n_tiles ? (n_tiles - first + step - 1) / step : 0;
    if (tid == 0) {
        for (int s = 0; s < S && (size_t)s < my_tiles; ++s) {
            mbar_expect_tx(&full[s], TILE);
            bulk_g2s(smem + (size_t)s * TILE, base + (first + (size_t)s * step) * TILE, TILE, &full[s]);
        }
    }
    float acc = 0.f;
    bool dead = false;
    for (size_t it = 0; it < my_tiles; ++it) {
        const int s = (int)(it % S);
        const uint32_t parity = (uint32_t)((it / S) & 1);
        int spins = 0;
        bool ok = true;
        while (!mbar_try_wait(&full[s], parity)) {
            if (++spins > (1 << 20)) { ok = false; break; }
        }
        if (__syncthreads_or(!ok)) {  // uniform decision: nobody is left behind at a barrier
            dead = true;
            if (tid == 0) atomicExch(err, 1);
            break;
        }
        const float4* p = reinterpret_cast<const float4*>(smem + (size_t)s * TILE);
#pragma unroll 4
        for (int i = tid; i < TILE / 16; i += blockDim.x) { float4 t = p[i]; acc += t.x + t.y + t.z + t.w; }
        __syncthreads();
        if (tid == 0 && it + S < my_tiles) {
            mbar_expect_tx(&full[s], TILE);
            bulk_g2s(smem + (size_t)s * TILE, base + (first + (it + S) * step) * TILE, TILE, &full[s]);
        }
    }
    // if a wait gave up, copies may still be in flight: wait (bounded) for the stages that were issued
    if (dead && tid == 0) {
        for (int s = 0; s < S; ++s)
            for (int spins = 0; spins < (1 << 16); ++spins)
                if (mbar_try_wait(&full[s], 0) || mbar_try_wait(&full[s], 1)) break;
    }
    if (acc == 1234.5678f) sink[tid] = acc;
}

template <typename F>
float time_ms(F f, int reps) {
    cudaEvent_t a, b;
    CK(cudaEventCreate(&a)); CK(cudaEventCreate(&b));
    for (int i = 0; i < 3; ++i) f();
    CK(cudaDeviceSynchronize());
    CK(cudaEventRecord(a));
    for (int i = 0; i < reps; ++i) f();
    CK(cudaEventRecord(b));
    CK(cudaEventSynchronize(b));
    CK(cudaGetLastError());
    float ms; CK(cudaEventElapsedTime(&ms, a, b));
    return ms / reps;
}

int main(int argc, char** argv) {
    const size_t GB = 1ull << 30;
    const size_t gib = argc > 1 ? (size_t)atoi(argv[1]) : 8;
    if (gib < 1 || gib > 64) { printf("usage: bw_probe [GiB of device memory to stream, 1..64]\n"); return 2; }
    const size_t bytes = gib * GB;  // 8 GiB = 64x the L2
    char* buf; float* sink; int* err;
    CK(cudaMalloc(&buf, bytes)); CK(cudaMalloc(&sink, 4096)); CK(cudaMalloc(&err, 4));
    CK(cudaMemset(buf, 0, bytes)); CK(cudaMemset(err, 0, 4));
    int sms; CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
    const int reps = 10;
    auto report = [&](const char* name, float ms, double b) { printf("%-34s %8.3f ms  %8.1f GB/s\n", name, ms, b / ms / 1e6); fflush(stdout); };

    {   // 128-bit, K streams emulating M+2 read streams
        const size_t nv = bytes / 16;
#define R128(K, U, G) { size_t sv = nv / K; float ms = time_ms([&] { read128<K, U><<<sms * G, 256>>>((const float4*)buf, sv, sv, sink); }, reps); \
            char nm[64]; snprintf(nm, 64, "read128 K=%d U=%d grid=%dxSM", K, U, G); report(nm, ms, (double)sv * K * 16); }
        R128(1, 8, 8) R128(1, 16, 4) R128(4, 4, 8) R128(8, 2, 8) R128(8, 2, 64) R128(8, 4, 4) R128(16, 1, 8) R128(16, 2, 64) R128(16, 2, 4)
    }
    {   // 256-bit
        const size_t nv = bytes / 32;
#define R256(K, U, G) { size_t sv = nv / K; float ms = time_ms([&] { read256<K, U><<<sms * G, 256>>>((const F8*)buf, sv, sv, sink); }, reps); \
            char nm[64]; snprintf(nm, 64, "read256 K=%d U=%d grid=%dxSM", K, U, G); report(nm, ms, (double)sv * K * 32); }
        R256(1, 4, 8) R256(1, 8, 4) R256(4, 2, 8) R256(8, 1, 8) R256(8, 2, 4) R256(8, 2, 64) R256(16, 1, 64)
    }
    {   // copy
        const size_t nv = bytes / 32;  // half src half dst
        float ms = time_ms([&] { copy128<4><<<sms * 8, 256>>>((const float4*)buf, (float4*)(buf + bytes / 2), nv); }, reps);
        report("copy128 U=4 grid=8xSM (r+w bytes)", ms, (double)nv * 32);
        ms = time_ms([&] { copy128<8><<<sms * 64, 256>>>((const float4*)buf, (float4*)(buf + bytes / 2), nv); }, reps);
        report("copy128 U=8 grid=64xSM (r+w bytes)", ms, (double)nv * 32);
        ms = time_ms([&] { CK(cudaMemcpyAsync(buf + bytes / 2, buf, bytes / 2, cudaMemcpyDeviceToDevice)); }, reps);
        report("cudaMemcpy D2D (r+w bytes)", ms, (double)bytes);
    }
    {   // TMA bulk
#define RTMA(TILE, S, G, T) { size_t nt = bytes / TILE; CK(cudaFuncSetAttribute(read_tma<TILE, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, TILE * S)); \
            float ms = time_ms([&] { read_tma<TILE, S><<<sms * G, T, TILE * S>>>(buf, nt, sink, err); }, reps); \
            char nm[64]; snprintf(nm, 64, "tma TILE=%d S=%d grid=%dxSM T=%d", TILE, S, G, T); report(nm, ms, (double)nt * TILE); \
            int h; CK(cudaMemcpy(&h, err, 4, cudaMemcpyDeviceToHost)); if (h) { printf("  (a wait gave up)\n"); CK(cudaMemset(err, 0, 4)); } }
        RTMA(16384, 4, 3, 128) RTMA(16384, 8, 1, 256) RTMA(8192, 8, 3, 128) RTMA(32768, 6, 1, 256) RTMA(16384, 12, 1, 256) RTMA(8192, 6, 4, 128)
    }
    CK(cudaFree(buf)); CK(cudaFree(sink)); CK(cudaFree(err));
    return 0;
}
