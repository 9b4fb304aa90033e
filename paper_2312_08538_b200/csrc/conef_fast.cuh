// Tuned kernels for large, aligned tensors (placeholder: everything falls back
// to the generic kernels).
#pragma once
#include <vector>

#include "conef_internal.h"

namespace conef {

inline void fast_classify(LayerDesc &L, int ckind, int unit)
{
    (void)ckind;
    (void)unit;
    L.fast = 0;
}
// return 1: not handled, the caller runs the generic kernel
inline int fast_pass1(int64_t &, const std::vector<LayerDesc> &, const DevView &, int, cudaStream_t) { return 1; }
inline int fast_pass2(int64_t &, const std::vector<LayerDesc> &, const DevView &, int, cudaStream_t) { return 1; }
inline int fast_pass3(int64_t &, const std::vector<LayerDesc> &, const DevView &, int, cudaStream_t) { return 1; }
inline int fast_gram_schmidt(int64_t &, const std::vector<LayerDesc> &, const DevView &, float *, cudaStream_t) { return 1; }

}  // namespace conef
