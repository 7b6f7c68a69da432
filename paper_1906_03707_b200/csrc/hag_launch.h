// Host-side helpers shared by the .cu files of the library: device selection for the span of a call,
// the launch with programmatic stream serialisation that every kernel uses, and two small predicates.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

namespace hagl {

// Makes `device` current for the lifetime of the object and restores the previous device afterwards.
struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

// Every kernel is launched with programmatic stream serialisation (see hag_kernels.cuh).
template <typename Args>
cudaError_t launch_pdl(void (*kernel)(Args), unsigned grid, unsigned threads, const Args &args, cudaStream_t s) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args);
}

// Lanes that cover one row with one 16-byte load each: the power of two >= the row's 16-byte chunks, 4..32.
inline int lanes_per_row(int n_chunks) {
    int l = 4;
    while (l < 32 && l < n_chunks) l *= 2;
    return l;
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace hagl
