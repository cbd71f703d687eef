// The library context behind the opaque reader_ctx handle.
#pragma once
#include "common.cuh"
#include "verify_attn_sm100.cuh"

struct reader_ctx {
    int device;
    int n_sm;
    int attn_kernel;  // 0 auto, 1 generic (CUDA cores), 2 tensor-core kernel only
    reader::Sm100Host sm100;
    cudaEvent_t ev_start, ev_stop;  // optional timing hooks around the main attention kernel
    cudaEvent_t ev_acc_start, ev_acc_stop;  // and around the argmax kernel of reader_accept
};
