// Stage 2b: candidate documents of a query = every document that owns a token in one of the probed posting lists
// (Sec. 3.2 step 1: L_q is the union of the probed lists, S the set of their source documents).
//
// The inverted file stores, per centroid, the unique ids of those documents.  Each probed list is streamed once and
// sets one bit per document in a per-query bitmap (the dedup); the bitmap is then compacted into an ascending id
// list with a three-kernel count / scan / write pass.
#include "common.cuh"

namespace chimera {

// grid (nq * P, B): one block per probed list.
__global__ void __launch_bounds__(128)
mark_kernel(const int32_t *__restrict__ probes, int n_lists, const int64_t *__restrict__ ivf_off,
            const int32_t *__restrict__ ivf_doc, uint32_t *__restrict__ bitmap, int64_t words)
{
    const int b = blockIdx.y;
    const int32_t c = DBG_CID(probes[(int64_t)b * n_lists + blockIdx.x]);
    uint32_t *bm = bitmap + (int64_t)b * words;
    const int64_t lo = ivf_off[c], hi = ivf_off[c + 1];
    // four list entries per thread and iteration: their loads and the bitmap reads they lead to are in flight together
    for (int64_t e0 = lo + threadIdx.x; e0 < hi; e0 += 4 * (int64_t)blockDim.x) {
        uint32_t d[4], cur[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t e = e0 + u * (int64_t)blockDim.x;
            d[u] = e < hi ? (uint32_t)ivf_doc[e] : 0xffffffffu;
            if (e < hi && !DBG_DOC_OK(d[u])) d[u] = 0xffffffffu;          // (debug build) skip a bad list entry
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) cur[u] = d[u] != 0xffffffffu ? bm[d[u] >> 5] : 0xffffffffu;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t bit = 1u << (d[u] & 31);
            if (!(cur[u] & bit)) atomicOr(&bm[d[u] >> 5], bit);
        }
    }
}

constexpr int CHUNK_THREADS = 256;
constexpr int WORDS_PER_THREAD = BITMAP_CHUNK_WORDS / CHUNK_THREADS;   // 4 consecutive words per thread
constexpr int COMPACT_STAGE = 8192;      // ids a chunk stages in shared memory (a chunk covers 32,768 documents)

__device__ __forceinline__ int block_exclusive_scan_256(int v, int *total)
{
    __shared__ int warp_part[CHUNK_THREADS / 32];
    int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_part[warp] = incl;
    __syncthreads();
    int before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < CHUNK_THREADS / 32; ++w) {
        int pw = warp_part[w];
        if (w < warp) before += pw;
        all += pw;
    }
    *total = all;
    return before + incl - v;
}

// grid (n_chunks, B): number of set bits in each chunk -> chunk_cnt[b][chunk].
__global__ void __launch_bounds__(CHUNK_THREADS)
count_kernel(const uint32_t *__restrict__ bitmap, int64_t words, int n_chunks, int32_t *__restrict__ chunk_cnt)
{
    const int b = blockIdx.y;
    const uint32_t *bm = bitmap + (int64_t)b * words;
    int64_t w0 = (int64_t)blockIdx.x * BITMAP_CHUNK_WORDS + threadIdx.x * WORDS_PER_THREAD;
    int c = 0;
#pragma unroll
    for (int j = 0; j < WORDS_PER_THREAD; ++j)
        if (w0 + j < words) c += __popc(bm[w0 + j]);
    int total;
    block_exclusive_scan_256(c, &total);
    if (threadIdx.x == 0) chunk_cnt[(int64_t)b * (n_chunks + 1) + blockIdx.x] = total;
}

// grid (B), one warp: exclusive scan of the chunk counts in place; entry n_chunks and n_cand[b] get the total
// (clamped to maxc; an overflow sets the status bit).
__global__ void __launch_bounds__(32)
chunk_scan_kernel(int32_t *__restrict__ chunk_cnt, int n_chunks, int64_t maxc, int32_t *__restrict__ n_cand,
                  uint32_t *status)
{
    const int b = blockIdx.x, lane = threadIdx.x;
    int32_t *cc = chunk_cnt + (int64_t)b * (n_chunks + 1);
    int run = 0;
    for (int base = 0; base < n_chunks; base += 32) {
        int i = base + lane;
        int v = i < n_chunks ? cc[i] : 0;
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (i < n_chunks) cc[i] = run + incl - v;
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) {
        cc[n_chunks] = run;
        if ((int64_t)run > maxc) {
            atomicOr(status, ST_OVERFLOW);
            run = (int)maxc;
        }
        n_cand[b] = run;
    }
}

// grid (n_chunks, B): write the ids of the set bits of each chunk, ascending, at its scanned offset.
__global__ void __launch_bounds__(CHUNK_THREADS)
compact_kernel(const uint32_t *__restrict__ bitmap, int64_t words, int n_chunks,
               const int32_t *__restrict__ chunk_cnt, int64_t maxc, int32_t *__restrict__ cand,
               int32_t *__restrict__ word_rank)
{
    const int b = blockIdx.y;
    const uint32_t *bm = bitmap + (int64_t)b * words;
    int64_t w0 = (int64_t)blockIdx.x * BITMAP_CHUNK_WORDS + threadIdx.x * WORDS_PER_THREAD;
    uint32_t w[WORDS_PER_THREAD];
    int c = 0;
#pragma unroll
    for (int j = 0; j < WORDS_PER_THREAD; ++j) {
        w[j] = (w0 + j < words) ? bm[w0 + j] : 0u;
        c += __popc(w[j]);
    }
    int total;
    const int local = block_exclusive_scan_256(c, &total);
    const int64_t base = chunk_cnt[(int64_t)b * (n_chunks + 1) + blockIdx.x];
    int32_t *out = cand + (int64_t)b * maxc;
    // A thread's ids are consecutive in the output but the threads' runs are ~30 ids apart, so direct stores are
    // scattered 4-byte writes: when the chunk's ids fit, they are staged in shared memory and copied out coalesced.
    __shared__ int32_t staged[COMPACT_STAGE];
    const bool use_stage = total <= COMPACT_STAGE;
    int64_t pos = use_stage ? local : base + local;
#pragma unroll
    for (int j = 0; j < WORDS_PER_THREAD; ++j) {
        uint32_t bits = w[j];
        if (w0 + j < words)
            word_rank[(int64_t)b * words + w0 + j] = (int32_t)(use_stage ? base + pos : pos);
        while (bits) {
            int t = __ffs(bits) - 1;
            bits &= bits - 1;
            const int32_t id = (int32_t)(((w0 + j) << 5) + t);
            if (use_stage) staged[pos] = id;
            else if (pos < maxc) out[pos] = id;
            ++pos;
        }
    }
    if (use_stage) {
        __syncthreads();
        for (int e = threadIdx.x; e < total; e += CHUNK_THREADS)
            if (base + e < maxc) out[base + e] = staged[e];
    }
}

int launch_gather(const Index &ix, const Params &p, const Layout &L, const int32_t *probes, uint32_t *bitmap,
                  int32_t *chunk_cnt, int32_t *cand, int32_t *n_cand, int32_t *word_rank, uint32_t *status,
                  cudaStream_t st)
{
    CHIMERA_CUDA(cudaMemsetAsync(bitmap, 0, sizeof(uint32_t) * (size_t)L.words * p.B, st));
    const int n_lists = p.nq * p.P;
    mark_kernel<<<dim3((unsigned)n_lists, (unsigned)p.B), 128, 0, st>>>(probes, n_lists, ix.ivf_off, ix.ivf_doc,
                                                                         bitmap, L.words);
    CHIMERA_CUDA(cudaGetLastError());
    dim3 gc((unsigned)L.n_chunks, (unsigned)p.B);
    count_kernel<<<gc, CHUNK_THREADS, 0, st>>>(bitmap, L.words, L.n_chunks, chunk_cnt);
    CHIMERA_CUDA(cudaGetLastError());
    chunk_scan_kernel<<<(unsigned)p.B, 32, 0, st>>>(chunk_cnt, L.n_chunks, p.maxc, n_cand, status);
    CHIMERA_CUDA(cudaGetLastError());
    compact_kernel<<<gc, CHUNK_THREADS, 0, st>>>(bitmap, L.words, L.n_chunks, chunk_cnt, p.maxc, cand, word_rank);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_GATHER, 4);
    return CHIMERA_OK;
}

}  // namespace chimera
