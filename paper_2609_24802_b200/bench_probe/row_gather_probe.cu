// Measurement probe of the benchmark (not part of libtiga.so, no counterpart in the paper):
// index-driven row gathers with the access shape of the stored-relation forward -- one row per
// group of LN lanes, 128-bit loads, four rows in flight per lane -- folded into one number so
// that nothing is optimised away.  The benchmark times it on a table that fits L2 to obtain the
// L2 -> SM gather bandwidth that bounds the forward when the gathered rows are cache resident,
// and on a workload's own index stream to obtain the time of its gathers alone.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

template <int LN>
__global__ void __launch_bounds__(256) row_gather_probe_kernel(const uint4* __restrict__ table, const int32_t* __restrict__ idx,
                                                               long long n_idx, float* sink) {
    const int ln = threadIdx.x % LN;
    const long long groups = (long long)gridDim.x * (blockDim.x / LN);
    const long long g0 = (long long)blockIdx.x * (blockDim.x / LN) + threadIdx.x / LN;
    float acc = 0.f;
    for (long long k = g0 * 4; k < n_idx; k += groups * 4) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long kk = k + u < n_idx ? k + u : k;
            v[u] = __ldg(table + (unsigned long long)(unsigned)__ldg(idx + kk) * LN + ln);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) acc += __uint_as_float(v[u].x) + __uint_as_float(v[u].y) + __uint_as_float(v[u].z) + __uint_as_float(v[u].w);
    }
    if (acc == 123.456f) atomicAdd(sink, acc);      // keeps the loads alive; practically never taken
}

}  // namespace

// table: device, n_rows rows of row_bytes bytes (16, 32, 64, 128, 256 or 512), 16-byte aligned;
// idx: device int32 [n_idx], every entry in [0, n_rows); sink: device fp32 [1]; stream: cudaStream_t.
// Returns 0 on success, 1 for a bad argument, 2 for an unsupported row size, 4 for a CUDA error.
extern "C" int tiga_bench_probe_row_gather(const void* table, int64_t n_rows, int32_t row_bytes,
                                           const int32_t* idx, int64_t n_idx, float* sink, void* stream) {
    if (!table || !idx || !sink || n_rows <= 0 || n_idx < 0 || (reinterpret_cast<uintptr_t>(table) & 15u)) return 1;
    if (row_bytes < 16 || row_bytes > 512 || (row_bytes & 15)) return 1;
    const int ln = row_bytes / 16;
    if (ln & (ln - 1)) return 2;
    if (n_idx == 0) return 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const unsigned blocks = 148 * 8;
    const uint4* t = static_cast<const uint4*>(table);
    switch (ln) {
        case 1: row_gather_probe_kernel<1><<<blocks, 256, 0, s>>>(t, idx, n_idx, sink); break;
        case 2: row_gather_probe_kernel<2><<<blocks, 256, 0, s>>>(t, idx, n_idx, sink); break;
        case 4: row_gather_probe_kernel<4><<<blocks, 256, 0, s>>>(t, idx, n_idx, sink); break;
        case 8: row_gather_probe_kernel<8><<<blocks, 256, 0, s>>>(t, idx, n_idx, sink); break;
        case 16: row_gather_probe_kernel<16><<<blocks, 256, 0, s>>>(t, idx, n_idx, sink); break;
        default: row_gather_probe_kernel<32><<<blocks, 256, 0, s>>>(t, idx, n_idx, sink); break;
    }
    return cudaPeekAtLastError() == cudaSuccess ? 0 : 4;
}
