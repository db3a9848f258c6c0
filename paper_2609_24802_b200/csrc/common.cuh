// Shared host/device helpers of libtiga (CUDA side only; the CPU oracle shares nothing with this).
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include "tiga.h"

namespace tiga {

#define TIGA_CUDA_TRY(expr)                                   \
    do {                                                      \
        cudaError_t _e = (expr);                              \
        if (_e != cudaSuccess) return TIGA_ERR_CUDA;          \
    } while (0)

// Peek (do not clear sticky errors of other users of the context) after a launch.
static inline tiga_status launch_status() {
    return cudaPeekAtLastError() == cudaSuccess ? TIGA_OK : TIGA_ERR_CUDA;
}

// Every kernel launch of the library goes through counted(): the grid size passes through unchanged
// and the process-wide launch counter (read by tiga_kernel_launches) goes up by one.
void note_launch();
template <typename T>
static inline T counted(T grid) { note_launch(); return grid; }

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// A bump allocator over the caller's workspace (256-byte granules).
struct Carver {
    char* base;
    size_t off;
    explicit Carver(void* p) : base(static_cast<char*>(p)), off(0) {}
    template <typename T>
    T* take(size_t count) {
        T* r = reinterpret_cast<T*>(base + off);
        off += align_up(count * sizeof(T), 256);
        return r;
    }
};

// Checked build (-DTIGA_CHECKED, libtiga_checked.so): every index that is about to address a gathered row,
// an edge or a point is range-checked first; a violation sets a bit of a status word (one word per
// translation unit, read through tiga_checked_status) and the access goes to element 0 instead.  Nothing
// traps, so the context stays usable.  In the normal build checked() is the identity.
enum : unsigned { CHECK_SOURCE = 1u, CHECK_EDGE = 2u, CHECK_POINT = 4u, CHECK_SLOT = 8u };
#ifdef TIGA_CHECKED
static __device__ unsigned int g_check_status;
template <typename I>
__device__ __forceinline__ I checked(I idx, long long n, unsigned code) {
    if ((long long)idx < 0 || (long long)idx >= n) { atomicOr(&g_check_status, code); return I(0); }
    return idx;
}
static inline unsigned read_check_status(bool reset) {
    unsigned v = 0, z = 0;
    if (cudaMemcpyFromSymbol(&v, g_check_status, sizeof(v)) != cudaSuccess) return 0x80000000u;
    if (reset) cudaMemcpyToSymbol(g_check_status, &z, sizeof(z));
    return v;
}
#else
template <typename I>
__device__ __forceinline__ I checked(I idx, long long, unsigned) { return idx; }
static inline unsigned read_check_status(bool) { return 0u; }
#endif
// one reader per translation unit (defined at the end of every .cu file), combined by tiga_checked_status
unsigned check_status_csr(bool reset);
unsigned check_status_csr_plan(bool reset);
unsigned check_status_csr_attention(bool reset);
unsigned check_status_radius(bool reset);
unsigned check_status_radius_lj(bool reset);
unsigned check_status_radius_mlp(bool reset);
unsigned check_status_knn(bool reset);

// streaming (read-once) loads and write-once stores keep L2 for the gathered rows
template <typename T>
__device__ __forceinline__ T ld_stream(const T* p) { return __ldcs(p); }
template <typename T>
__device__ __forceinline__ void st_stream(T* p, T v) { __stcs(p, v); }

}  // namespace tiga
