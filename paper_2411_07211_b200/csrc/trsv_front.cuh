// Interface between the trsv entry points and the sub-block kernel (trsv_front.cu).
#pragma once
#include "common.cuh"

namespace b2 {

// Tries the sub-block kernel.  Returns a status; *handled is false (and nothing was launched)
// when the call does not meet the kernel's preconditions (16-byte aligned matrix, lda a
// multiple of the pack length, workspace large enough) -- the caller then uses the general
// block-row kernel.  `xbase` is the vector base per vec_base().
template <typename T>
int trsv_front_try(const Launch& l, bool coltype, bool backward, bool unit, int64_t n, const T* a, int64_t lda,
                   T* xbase, int64_t incx, unsigned tag, bool* handled);

}  // namespace b2
