// Document-sharded search (the scaling sketch of Sec. 3.3: each GPU holds a slice of the documents, only ids and
// scores move between GPUs): the small kernels around the exchange steps.  The selections themselves are
// shard_select_kernel (next to select_kernel, whose radix select it shares) and the top-k kernels.
#include <limits.h>

#include "common.cuh"

namespace chimera {

// A shard's local top-n_prune list for the exchange: global ids (local id + doc_base; -1 stays) and their scores.
__global__ void shard_export_kernel(const int32_t *__restrict__ pruned, const int32_t *__restrict__ pruned_ci, int64_t n,
                                    long long doc_base, int32_t *__restrict__ out_ids, int32_t *__restrict__ out_ci)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        const int32_t d = pruned[i];
        out_ids[i] = d >= 0 ? (int32_t)(d + doc_base) : -1;
        out_ci[i] = d >= 0 ? pruned_ci[i] : INT_MIN;
    }
}

__global__ void add_base_kernel(int32_t *__restrict__ ids, int64_t n, long long doc_base)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n && ids[i] >= 0) ids[i] = (int32_t)(ids[i] + doc_base);
}

int launch_shard_export(const Params &p, const int32_t *pruned, const int32_t *pruned_ci, int64_t doc_base,
                        int32_t *out_ids, int32_t *out_ci, cudaStream_t st)
{
    const int64_t n = (int64_t)p.B * p.n_prune;
    shard_export_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(pruned, pruned_ci, n, (long long)doc_base, out_ids,
                                                                     out_ci);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_MISC);
    return CHIMERA_OK;
}

int launch_add_base(int32_t *ids, int64_t n, int64_t doc_base, cudaStream_t st)
{
    add_base_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(ids, n, (long long)doc_base);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_MISC);
    return CHIMERA_OK;
}

}  // namespace chimera
