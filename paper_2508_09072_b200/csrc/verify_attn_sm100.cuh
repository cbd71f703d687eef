// Host-side interface of the tensor-core (tcgen05 + TMA) verify-attention kernel.
#pragma once
#include "common.cuh"

namespace reader {

struct Sm100Host {
    void *encode_tiled;   // cuTensorMapEncodeTiled, resolved through the runtime (no libcuda link)
    int smem_optin;       // opt-in shared memory per block on the device
    bool ready;
};

reader_status sm100_host_init(Sm100Host *h, int device);
bool sm100_supports(const Sm100Host *h, const AttnParams &p);
reader_status launch_attn_sm100(const Sm100Host *h, const AttnParams &p, const reader_kv_cache &cache,
                                cudaStream_t st);

}  // namespace reader
