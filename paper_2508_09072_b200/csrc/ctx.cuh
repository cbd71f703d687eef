// The library context behind the opaque reader_ctx handle.
#pragma once
#include "common.cuh"
#include "verify_attn_sm100.cuh"

// What reader_verify_prepare left in a workspace, so that reader_verify_attn_prepared can tell whether it is
// being called for the same problem.
struct PreparedRecord {
    bool valid;
    const void *workspace, *page_table, *seq_lens, *parent, *anc_mask;
    int32_t *status;
    int B, T, Hq, Hkv, D, max_pages, num_pages, shared_prefix_len;
};

struct reader_ctx {
    int device;
    int n_sm;
    int attn_kernel;  // 0 auto, 1 generic (CUDA cores), 2 tensor-core kernel only
    int partition;    // 0 auto, 1 equal ranges, 2 aligned whenever a prefix is shared
    reader::Sm100Host sm100;
    cudaEvent_t ev_start, ev_stop;  // optional timing hooks around the main attention kernel
    cudaEvent_t ev_acc_start, ev_acc_stop;  // and around the argmax kernel of reader_accept
    PreparedRecord prepared;
};
