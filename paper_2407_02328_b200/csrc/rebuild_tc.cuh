// Tensor-core (tcgen05) rebuild projection for bfloat16 caches.
#pragma once

#include <vector>

#include "../../include/adore.h"
#include "rebuild_simt.cuh"

namespace adore {

struct TcState { bool ready = false; };

template <typename T> inline bool tc_usable(const TcState&) { return false; }
inline adore_status_t tc_init(TcState&, const adore_config_t&, std::vector<void*>&, cudaStream_t) { return ADORE_OK; }
inline adore_status_t tc_set_weights(TcState&, int, const void*) { return ADORE_OK; }
template <typename T>
inline cudaError_t launch_rebuild_tc(TcState&, const RebuildParams<T>&, int, int, cudaStream_t, int*) { return cudaErrorNotSupported; }

}  // namespace adore
