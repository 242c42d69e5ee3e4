// Shared between the host-only and the CUDA translation units of the library.
#ifndef PREBA_INTERNAL_H_
#define PREBA_INTERNAL_H_

#include <stdint.h>

#include "preba.h"

namespace preba {

bool dtype_ok(int out_dtype);
uint32_t dtype_bytes(int out_dtype);  // size of one output element
bool dims_ok(uint32_t h, uint32_t w);
uint64_t align_up(uint64_t v, uint64_t a);

// The cudaError_t behind the calling thread's last PREBA_ERR_CUDA (preba_last_cuda_error).
extern thread_local int g_last_cuda_error;

}  // namespace preba

#endif  // PREBA_INTERNAL_H_
