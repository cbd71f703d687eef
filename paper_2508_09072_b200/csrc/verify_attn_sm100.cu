// Tensor-core verify attention for sm_100a (placeholder until the tcgen05 kernel lands).
#include "verify_attn_sm100.cuh"

namespace reader {

reader_status sm100_host_init(Sm100Host *h, int) {
    h->encode_tiled = nullptr;
    h->smem_optin = 0;
    h->ready = false;
    return READER_OK;
}
bool sm100_supports(const Sm100Host *, const AttnParams &) { return false; }
reader_status launch_attn_sm100(const Sm100Host *, const AttnParams &, const reader_kv_cache &, cudaStream_t) {
    return READER_ERR_UNSUPPORTED;
}

}  // namespace reader
