// reader_accept_noalloc: the acceptance step for callers that cannot hand over scratch memory.
//
// reader_accept splits every logits row across several thread blocks and parks the per-block
// (maximum, index) pairs in the caller's workspace before the walk kernel reduces them.  Some
// hosts have nowhere to get such a workspace from at the moment they call: a serving process
// whose whole device memory was handed to another allocator at start-up (cudaMalloc then fails
// or stalls every stream while it synchronises the device), or a decode loop that has promised
// its scheduler to make no allocating call between steps.  For them the same two kernels run
// with the pairs parked in a fixed array that is part of this library's device image.
//
// What that means for the user:
//   * the array occupies kScratchBytes (2 MiB) on every GPU that loads the library, until the
//     process ends;
//   * problems with batch * n_nodes above READER_NOALLOC_MAX_ROWS are refused
//     (READER_ERR_TOO_LARGE), nothing is launched;
//   * the first call on a device looks the array's device address up (one runtime query, no
//     allocation) and remembers it; make that first call outside any stream capture;
//   * all calls share the one array and each leaves its pairs behind.  Nothing has to start at
//     zero: every slot the walk kernel reads is written by the scan kernel of the same call
//     first.  Two calls that may run on the GPU at the same time (different streams) would
//     overwrite each other's pairs: keep them on one stream or order them yourself.
#include <mutex>

#include "common.cuh"
#include "ctx.cuh"

namespace {

constexpr int kMaxRows = READER_NOALLOC_MAX_ROWS;
constexpr int kSplitsCap = reader::kMaxArgmaxSplits;   // the array holds that many pairs per row
constexpr size_t kScratchBytes = (size_t)kMaxRows * kSplitsCap * (sizeof(float) + sizeof(int32_t));

// Device-side storage.  In host code this name is only a handle for the runtime's symbol lookup,
// never a pointer a kernel could use: the address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_scratch_addr[kMaxDevices];   // per device, filled on the first call there

// The calling thread's current device must be `device`.
reader_status scratch_for_device(int device, unsigned char **out) {
    if (device < 0 || device >= kMaxDevices) return READER_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[device]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return READER_ERR_CUDA;
        }
        g_scratch_addr[device] = p;
    }
    *out = static_cast<unsigned char *>(g_scratch_addr[device]);
    return READER_OK;
}

}  // namespace

extern "C" reader_status reader_accept_noalloc(reader_ctx *ctx, const reader_tree *tree, const int32_t *node_tokens,
                                               const float *logits, int32_t vocab, int32_t *target_ids,
                                               int32_t max_path, int32_t *path_out, int32_t *n_acc_out,
                                               int32_t *bonus_out, int32_t *status_out, void *stream) {
    using namespace reader;
    if (!ctx || !tree) return READER_ERR_INVALID_ARG;
    if (tree->batch == 0) return READER_OK;
    if (!tree->parent || !node_tokens || !logits || !target_ids || !path_out || !n_acc_out || !bonus_out || !status_out)
        return READER_ERR_INVALID_ARG;
    const int B = tree->batch, T = tree->n_nodes;
    if (B < 0 || T < 1 || T > kMaxNodes || max_path < 1 || vocab < 1 ||
        (reinterpret_cast<uintptr_t>(logits) & 15u) != 0)
        return READER_ERR_INVALID_ARG;
    const int64_t rows = (int64_t)B * T;
    if (rows > kMaxRows) return READER_ERR_TOO_LARGE;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return READER_ERR_CUDA;
    if (dev != ctx->device) return READER_ERR_INVALID_ARG;
    unsigned char *scratch = nullptr;
    if (reader_status st = scratch_for_device(dev, &scratch)) return st;

    const int splits = argmax_splits(ctx->n_sm, rows, vocab);   // the same cut as reader_accept; <= kSplitsCap
    float *part_val = reinterpret_cast<float *>(scratch);
    int32_t *part_idx = reinterpret_cast<int32_t *>(scratch + (size_t)kMaxRows * kSplitsCap * sizeof(float));

    cudaStream_t st = (cudaStream_t)stream;
    launch_argmax(logits, rows, vocab, splits, part_val, part_idx, st);
    launch_accept(tree->parent, node_tokens, target_ids, B, T, max_path, part_val, part_idx, splits, path_out,
                  n_acc_out, bonus_out, status_out, st);
    return cudaGetLastError() == cudaSuccess ? READER_OK : READER_ERR_CUDA;
}
