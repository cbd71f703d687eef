// Host-side interface of the tensor-core (tcgen05 + TMA) verify-attention kernel.
#pragma once
#include "common.cuh"

namespace reader {

struct Sm100Maps;   // cached TMA descriptors of the pool last seen

struct Sm100Host {
    void *encode_tiled;   // cuTensorMapEncodeTiled, resolved through the runtime (no libcuda link)
    int smem_optin;       // opt-in shared memory per block on the device
    bool ready;           // the kernel can run on this device
    bool attr_set;        // dynamic shared memory limit raised (done on first launch, device current)
    Sm100Maps *maps;
};

reader_status sm100_host_init(Sm100Host *h, int device);
void sm100_host_destroy(Sm100Host *h);
bool sm100_supports(const Sm100Host *h, const AttnParams &p, float softmax_scale);
reader_status launch_attn_sm100(Sm100Host *h, const AttnParams &p, int small_cluster, cudaStream_t st);

}  // namespace reader
