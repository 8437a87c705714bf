// Memory-system probes: the denominators of the random-access roofline.
//   random read : independent uniformly random aligned granules (32 / 64 / 128 bytes), many in
//                 flight per thread, every SM full -> the rate HBM sustains for scattered sectors;
//   chase       : chains of dependent loads over a random cycle -> the latency one pointer-chasing
//                 chain pays per hop, alone or with many chains running side by side.
#include "common.h"

#include <algorithm>
#include <cstring>
#include <vector>

namespace {

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// LANES adjacent lanes read one granule of LANES * 16 bytes; each lane group issues `per_group`
// granule reads, UNROLL of them in flight at a time.
template <int LANES>
__global__ void random_read_kernel(const uint4* buf, uint64_t n_granules, int per_group, uint64_t salt,
                                   unsigned long long* sink) {
    constexpr int UNROLL = 8;
    const uint64_t tid = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x;
    const uint64_t group = tid / LANES;
    const int sub = (int)(tid % LANES);
    uint32_t acc = 0;
    for (int i = 0; i < per_group; i += UNROLL) {
        uint4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; u++) {
            uint64_t g = mix64(salt + group * 0x9E3779B97F4A7C15ull + (uint64_t)(i + u)) % n_granules;
            v[u] = __ldg(buf + g * LANES + sub);
        }
#pragma unroll
        for (int u = 0; u < UNROLL; u++) acc += v[u].x ^ v[u].w;
    }
    if (acc == 0x12345679u) atomicAdd(sink, 1ull);      // keeps the loads alive
}

__global__ void scatter_next_kernel(unsigned char* buf, const uint32_t* next, uint64_t n_lines) {
    uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x;
    if (i < n_lines) *reinterpret_cast<unsigned long long*>(buf + i * 128) = next[i];
}

// each block runs one chain with one thread; chain c starts at line starts[c]
__global__ void chase_kernel(const unsigned char* buf, const uint32_t* starts, long long hops,
                             unsigned long long* sink) {
    if (threadIdx.x != 0) return;
    unsigned long long p = starts[blockIdx.x];
    for (long long h = 0; h < hops; h++)
        p = *reinterpret_cast<const volatile unsigned long long*>(buf + p * 128);
    if (p == 0xFFFFFFFFFFFFull) atomicAdd(sink, 1ull);
}

}  // namespace

extern "C" int sam_probe_random_read(void* buf_dev, size_t footprint_bytes, int32_t granule, int32_t iters,
                                     void* stream, double* gbps, double* mreq_s) {
    if (!buf_dev || !gbps || !mreq_s || iters < 1 || footprint_bytes < (1u << 20)) return SAM_ERR_ARG;
    if (granule != 32 && granule != 64 && granule != 128) return SAM_ERR_ARG;
    if (((uintptr_t)buf_dev & 127) != 0) return SAM_ERR_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    int dev = 0, sms = 0;
    SAM_CUDA(cudaGetDevice(&dev));
    SAM_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    unsigned long long* sink = nullptr;
    SAM_CUDA(cudaMalloc(&sink, 8));
    cudaMemsetAsync(sink, 0, 8, s);
    const int threads = 256, blocks = sms * 8, per_group = 512;
    const int lanes = granule / 16;
    const uint64_t n_granules = footprint_bytes / (uint64_t)granule;
    const double requests = (double)blocks * threads / lanes * per_group;
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0); cudaEventCreate(&e1);
    float best = 1e30f;
    for (int it = 0; it <= iters; it++) {
        cudaEventRecord(e0, s);
        const uint64_t salt = 0xABCDEFull * (uint64_t)(it + 1);
        if (lanes == 2) random_read_kernel<2><<<blocks, threads, 0, s>>>((const uint4*)buf_dev, n_granules, per_group, salt, sink);
        else if (lanes == 4) random_read_kernel<4><<<blocks, threads, 0, s>>>((const uint4*)buf_dev, n_granules, per_group, salt, sink);
        else random_read_kernel<8><<<blocks, threads, 0, s>>>((const uint4*)buf_dev, n_granules, per_group, salt, sink);
        cudaEventRecord(e1, s);
        cudaError_t e = cudaEventSynchronize(e1);
        if (e != cudaSuccess) { sam_set_cuda_error(e); cudaFree(sink); return SAM_ERR_CUDA; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        if (it > 0 && ms < best) best = ms;              // launch 0 is the warm-up
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    cudaFree(sink);
    SAM_CUDA(cudaGetLastError());
    *gbps = requests * granule / (best * 1e-3) / 1e9;
    *mreq_s = requests / (best * 1e-3) / 1e6;
    return SAM_OK;
}

extern "C" int sam_probe_chase(void* buf_dev, size_t footprint_bytes, int64_t hops, int32_t chains,
                               void* stream, double* ns_per_hop) {
    if (!buf_dev || !ns_per_hop || hops < 1 || chains < 1 || chains > 65536) return SAM_ERR_ARG;
    if (footprint_bytes < (1u << 20) || ((uintptr_t)buf_dev & 127) != 0) return SAM_ERR_ARG;
    const uint64_t n_lines = footprint_bytes / 128;
    if (n_lines > 0xFFFFFFFFull || (uint64_t)chains > n_lines) return SAM_ERR_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    // Sattolo's algorithm: a uniformly random single cycle over the lines
    std::vector<uint32_t> next;
    std::vector<uint32_t> starts((size_t)chains);
    try { next.resize((size_t)n_lines); } catch (const std::bad_alloc&) { return SAM_ERR_NOMEM; }
    for (uint64_t i = 0; i < n_lines; i++) next[(size_t)i] = (uint32_t)i;
    uint64_t x = 0x853C49E6748FEA9Bull;
    for (uint64_t i = n_lines - 1; i > 0; i--) {
        x ^= x << 13; x ^= x >> 7; x ^= x << 17;
        uint64_t j = x % i;
        std::swap(next[(size_t)i], next[(size_t)j]);
    }
    for (int c = 0; c < chains; c++) starts[(size_t)c] = (uint32_t)((n_lines / (uint64_t)chains) * (uint64_t)c);
    uint32_t* d_next = nullptr; uint32_t* d_starts = nullptr; unsigned long long* sink = nullptr;
    cudaError_t e = cudaMalloc(&d_next, (size_t)n_lines * 4);
    if (e == cudaSuccess) e = cudaMalloc(&d_starts, (size_t)chains * 4);
    if (e == cudaSuccess) e = cudaMalloc(&sink, 8);
    if (e != cudaSuccess) { sam_set_cuda_error(e); cudaGetLastError(); cudaFree(d_next); cudaFree(d_starts); return SAM_ERR_NOMEM; }
    cudaMemcpyAsync(d_next, next.data(), (size_t)n_lines * 4, cudaMemcpyHostToDevice, s);
    cudaMemcpyAsync(d_starts, starts.data(), (size_t)chains * 4, cudaMemcpyHostToDevice, s);
    cudaMemsetAsync(sink, 0, 8, s);
    scatter_next_kernel<<<(unsigned)((n_lines + 255) / 256), 256, 0, s>>>((unsigned char*)buf_dev, d_next, n_lines);
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0); cudaEventCreate(&e1);
    chase_kernel<<<chains, 32, 0, s>>>((const unsigned char*)buf_dev, d_starts, hops / 8 + 1, sink);   // warm-up
    cudaEventRecord(e0, s);
    chase_kernel<<<chains, 32, 0, s>>>((const unsigned char*)buf_dev, d_starts, hops, sink);
    cudaEventRecord(e1, s);
    e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    cudaFree(d_next); cudaFree(d_starts); cudaFree(sink);
    if (e != cudaSuccess) { sam_set_cuda_error(e); return SAM_ERR_CUDA; }
    SAM_CUDA(cudaGetLastError());
    *ns_per_hop = (double)ms * 1e6 / (double)hops;
    return SAM_OK;
}
