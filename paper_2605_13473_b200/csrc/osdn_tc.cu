// tcgen05 / TMA kernels of the OSDN layer for bf16 I/O (sm_100a).
#include "osdn_common.cuh"

namespace osdn {

bool tc_supported(const osdn_params&) { return false; }

int tc_forward(const osdn_params&, const Hyper&, const WsLayout&, void*, const Pointers&, bool, cudaStream_t)
{
    return -1;
}

int tc_backward(const osdn_params&, const Hyper&, const WsLayout&, void*, const Pointers&, cudaStream_t)
{
    return -1;
}

}  // namespace osdn
