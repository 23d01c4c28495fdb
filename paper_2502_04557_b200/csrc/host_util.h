// Host-side helpers shared by the files that implement the C ABI: argument checks and workspace
// carving.
#pragma once

#include <stddef.h>
#include <stdint.h>

#include "launch.h"
#include "sprinter.h"

namespace spr {

inline bool dtype_ok(int dt) { return dt == SPR_F32 || dt == SPR_BF16; }
inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// typed pointer `off` bytes into the workspace
template <typename T>
inline T *at(void *ws, size_t off)
{
    return reinterpret_cast<T *>(static_cast<char *>(ws) + off);
}

// status of an entry point whose last CUDA call returned e
inline int finish(cudaError_t e) { return e == cudaSuccess ? SPR_OK : report_cuda_error(e); }

}  // namespace spr
