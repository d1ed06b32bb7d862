// Offline index construction on the device (Sec. 3.1: centroids, posting lists, per-token codes).
//   - prefix sums of the document lengths (token offset of each document)
//   - fixed-point digit planes of the centroids, the stationary operand of the score-table GEMM
//   - an inverted file: per centroid, the unique ids of the documents that own a token assigned to it
#include <stdio.h>

#include "common.cuh"

namespace chimera {

// ------------------------------------------------------------------------------------------------ validation ----
__global__ void validate_kernel(const int32_t *__restrict__ cids, int64_t T, int64_t K,
                                const int32_t *__restrict__ doclens, int64_t N, int32_t *flags, int32_t *max_len)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int bad_cid = 0, bad_len = 0, mx = 0;
    for (int64_t t = i; t < T; t += stride) {
        int32_t c = cids[t];
        if (c < 0 || c >= K) bad_cid = 1;
    }
    for (int64_t d = i; d < N; d += stride) {
        int32_t l = doclens[d];
        if (l < 1) bad_len = 1;
        mx = l > mx ? l : mx;
    }
    if (bad_cid) atomicOr(&flags[0], 1);
    if (bad_len) atomicOr(&flags[0], 2);
    if (mx > 0) atomicMax(max_len, mx);
}

// --------------------------------------------------------------------------------------- exclusive scan (i32->i64)
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 8;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

__global__ void scan_tile_sums(const int32_t *__restrict__ in, int64_t n, int64_t *__restrict__ tile_sum)
{
    __shared__ long long warp_part[SCAN_THREADS / 32];
    int64_t base = (int64_t)blockIdx.x * SCAN_TILE;
    long long s = 0;
    for (int j = 0; j < SCAN_ITEMS; ++j) {
        int64_t i = base + (int64_t)j * SCAN_THREADS + threadIdx.x;
        if (i < n) s += in[i];
    }
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long t = 0;
        for (int w = 0; w < SCAN_THREADS / 32; ++w) t += warp_part[w];
        tile_sum[blockIdx.x] = t;
    }
}

// One thread: exclusive scan of the tile sums in place; writes the grand total to out[n].
__global__ void scan_tile_offsets(int64_t *tile_sum, int64_t n_tiles, int64_t *out, int64_t n)
{
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        long long run = 0;
        for (int64_t i = 0; i < n_tiles; ++i) {
            long long v = tile_sum[i];
            tile_sum[i] = run;
            run += v;
        }
        out[n] = run;
    }
}

__global__ void scan_tiles(const int32_t *__restrict__ in, int64_t n, const int64_t *__restrict__ tile_off,
                           int64_t *__restrict__ out)
{
    __shared__ long long warp_part[SCAN_THREADS / 32];
    // thread owns SCAN_ITEMS consecutive elements
    int64_t first = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    long long v[SCAN_ITEMS];
    long long s = 0;
    for (int j = 0; j < SCAN_ITEMS; ++j) {
        v[j] = (first + j < n) ? in[first + j] : 0;
        s += v[j];
    }
    long long incl = s;
    int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int o = 1; o < 32; o <<= 1) {
        long long t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_part[warp] = incl;
    __syncthreads();
    long long before = 0;
    for (int w = 0; w < warp; ++w) before += warp_part[w];
    long long run = tile_off[blockIdx.x] + before + incl - s;
    for (int j = 0; j < SCAN_ITEMS; ++j) {
        if (first + j < n) out[first + j] = run;
        run += v[j];
    }
}

// out[0..n] = exclusive prefix sums of in[0..n-1] (out has n+1 entries); tmp holds ceil(n / SCAN_TILE) int64.
static int exclusive_scan(const int32_t *in, int64_t n, int64_t *out, int64_t *tmp, cudaStream_t st)
{
    int64_t tiles = (n + SCAN_TILE - 1) / SCAN_TILE;
    scan_tile_sums<<<(unsigned)tiles, SCAN_THREADS, 0, st>>>(in, n, tmp);
    scan_tile_offsets<<<1, 32, 0, st>>>(tmp, tiles, out, n);
    scan_tiles<<<(unsigned)tiles, SCAN_THREADS, 0, st>>>(in, n, tmp, out);
    CHIMERA_CUDA(cudaGetLastError());
    return CHIMERA_OK;
}

// ------------------------------------------------------------------------------------------------ digit planes ---
// X = rint(x * 2^22) split into balanced base-256 digits X = d0 + 256 d1 + 65536 d2, d0, d1 in [-128, 127],
// |d2| <= 64.  Planes have a fixed row pitch of DIGIT_PITCH (128) bytes, dimensions >= D are zero:
// plane p of row r, dimension d sits at dig[(p * rows + r) * 128 + d].
// Rows must also be (at most) unit-norm: later stages rely on |S_fx| <= 2^24 + 2^16, which holds when both factors
// have sum_d X[d]^2 <= 2^44 + 2^35 (norm <= 1 + 2^-10).  A longer row sets the same status bit as an element out of
// range.  A block of 256 threads holds two rows (one thread per padded dimension).
constexpr int DIGIT_PITCH = 128;
constexpr long long MAX_ROW_SQUARE_SUM = (1LL << 44) + (1LL << 35);

__global__ void digits_kernel(const float *__restrict__ x, int64_t rows, int D, int8_t *__restrict__ dig,
                              uint32_t *status)
{
    __shared__ unsigned long long row_sq[2];
    const int64_t n = rows * DIGIT_PITCH;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (threadIdx.x < 2) row_sq[threadIdx.x] = 0ull;
    __syncthreads();
    const int64_t r = i / DIGIT_PITCH;
    const int d = (int)(i % DIGIT_PITCH);
    int d0 = 0, d1 = 0, d2 = 0;
    unsigned long long sq = 0ull;
    if (i < n && d < D) {
        float v = x[r * D + d];
        if (!(fabsf(v) <= 1.0f)) {
            if (status) atomicOr(status, ST_BAD_QUERY);
            v = fminf(fmaxf(v, -1.0f), 1.0f);
            if (v != v) v = 0.f;
        }
        const int X = __float2int_rn(v * 4194304.0f);
        sq = (unsigned long long)((long long)X * X);
        d0 = ((X + 128) & 255) - 128;
        const int X1 = (X - d0) >> 8;
        d1 = ((X1 + 128) & 255) - 128;
        d2 = (X1 - d1) >> 8;
    }
    if (i < n) {
        dig[i] = (int8_t)d0;
        dig[n + i] = (int8_t)d1;
        dig[2 * n + i] = (int8_t)d2;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if ((threadIdx.x & 31) == 0 && sq) atomicAdd(&row_sq[threadIdx.x / DIGIT_PITCH], sq);
    __syncthreads();
    if (threadIdx.x < 2 && row_sq[threadIdx.x] > (unsigned long long)MAX_ROW_SQUARE_SUM && status)
        atomicOr(status, ST_BAD_QUERY);
}

int launch_digits(const float *x, int64_t rows, int D, int8_t *dig, uint32_t *status, cudaStream_t st)
{
    const int64_t n = rows * DIGIT_PITCH;
    digits_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(x, rows, D, dig, status);
    CHIMERA_CUDA(cudaGetLastError());
    return CHIMERA_OK;
}

// ------------------------------------------------------------------------------------------------ inverted file --
// One warp per document.  A token is its document's representative for centroid c if no earlier token of the same
// document has the same centroid.  Pass 0 counts representatives per centroid; pass 1 writes the document id into
// the centroid's list (order inside a list is whatever the atomics give: consumers only set bits).
template <int PASS>
__global__ void ivf_kernel(const int32_t *__restrict__ cids, const int64_t *__restrict__ doc_off, int64_t N,
                           int32_t *__restrict__ count, const int64_t *__restrict__ ivf_off,
                           int32_t *__restrict__ ivf_doc)
{
    int lane = threadIdx.x & 31;
    int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t d = warp; d < N; d += n_warps) {
        int64_t b = doc_off[d], e = doc_off[d + 1];
        for (int64_t t = b + lane; t < e; t += 32) {
            int32_t c = cids[t];
            bool first = true;
            for (int64_t u = b; u < t; ++u)
                if (cids[u] == c) { first = false; break; }
            if (first) {
                int32_t pos = atomicAdd(&count[c], 1);
                if (PASS == 1) ivf_doc[ivf_off[c] + pos] = (int32_t)d;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------ token lists ----
// Per centroid the ids of its tokens and their documents (the posting lists P_i of Sec. 3.2 step 1 as the paper keeps
// them: token level).  One warp per document; pass 0 counts, pass 1 writes through an atomic cursor.
template <int PASS>
__global__ void token_list_kernel(const int32_t *__restrict__ cids, const int64_t *__restrict__ doc_off, int64_t N,
                                  int32_t *__restrict__ count, const int64_t *__restrict__ tok_off,
                                  int32_t *__restrict__ tok_id, int32_t *__restrict__ tok_doc)
{
    int lane = threadIdx.x & 31;
    int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t d = warp; d < N; d += n_warps) {
        int64_t b = doc_off[d], e = doc_off[d + 1];
        for (int64_t t = b + lane; t < e; t += 32) {
            int32_t c = cids[t];
            int32_t pos = atomicAdd(&count[c], 1);
            if (PASS == 1) {
                tok_id[tok_off[c] + pos] = (int32_t)t;
                tok_doc[tok_off[c] + pos] = (int32_t)d;
            }
        }
    }
}

// out[0] = max_c (off[c + 1] - off[c])
__global__ void max_list_kernel(const int64_t *__restrict__ off, int64_t K, unsigned long long *__restrict__ out)
{
    unsigned long long m = 0;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < K; c += (int64_t)gridDim.x * blockDim.x) {
        const unsigned long long len = (unsigned long long)(off[c + 1] - off[c]);
        m = len > m ? len : m;
    }
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long t = __shfl_xor_sync(0xffffffffu, m, o);
        m = t > m ? t : m;
    }
    if ((threadIdx.x & 31) == 0) atomicMax(out, m);
}

int build_token_lists(Index &ix, cudaStream_t st)
{
    if (ix.tok_id) return CHIMERA_OK;
    if (ix.T > 0x7fffffffLL) return fail(CHIMERA_UNSUPPORTED, "token ids must fit int32");
    int32_t *count = nullptr;
    int64_t *tmp = nullptr;
    int64_t *off = nullptr;
    int32_t *ids = nullptr, *docs = nullptr;
    auto cleanup = [&](bool all) {
        cudaFree(count);
        cudaFree(tmp);
        if (all) { cudaFree(off); cudaFree(ids); cudaFree(docs); }
    };
#define TL_CUDA(call)                                                                        \
    do {                                                                                     \
        cudaError_t e__ = (call);                                                            \
        if (e__ != cudaSuccess) {                                                            \
            cleanup(true);                                                                   \
            return fail(CHIMERA_CUDA_ERROR, "%s: %s", #call, cudaGetErrorString(e__));      \
        }                                                                                    \
    } while (0)
    TL_CUDA(cudaMalloc(&count, sizeof(int32_t) * ix.K));
    TL_CUDA(cudaMalloc(&tmp, sizeof(int64_t) * ((ix.K + SCAN_TILE - 1) / SCAN_TILE + 1)));
    TL_CUDA(cudaMalloc(&off, sizeof(int64_t) * (ix.K + 1)));
    TL_CUDA(cudaMalloc(&ids, sizeof(int32_t) * ix.T));
    TL_CUDA(cudaMalloc(&docs, sizeof(int32_t) * ix.T));
    TL_CUDA(cudaMemsetAsync(count, 0, sizeof(int32_t) * ix.K, st));
    int64_t warps_wanted = ix.N < (int64_t)ix.sm_count * 64 ? ix.N : (int64_t)ix.sm_count * 64;
    unsigned blocks = (unsigned)((warps_wanted * 32 + 255) / 256);
    token_list_kernel<0><<<blocks, 256, 0, st>>>(ix.cids, ix.doc_off, ix.N, count, nullptr, nullptr, nullptr);
    TL_CUDA(cudaGetLastError());
    int rc = exclusive_scan(count, ix.K, off, tmp, st);
    if (rc) { cleanup(true); return rc; }
    TL_CUDA(cudaMemsetAsync(count, 0, sizeof(int32_t) * ix.K, st));
    token_list_kernel<1><<<blocks, 256, 0, st>>>(ix.cids, ix.doc_off, ix.N, count, off, ids, docs);
    TL_CUDA(cudaGetLastError());
    // the longest list (sizes the hashed score table of the refinement); tmp is free again: its first word holds it
    TL_CUDA(cudaMemsetAsync(tmp, 0, sizeof(int64_t), st));
    max_list_kernel<<<(unsigned)((ix.K + 255) / 256 < 1024 ? (ix.K + 255) / 256 : 1024), 256, 0, st>>>(
        off, ix.K, reinterpret_cast<unsigned long long *>(tmp));
    TL_CUDA(cudaGetLastError());
    long long longest = 0;
    TL_CUDA(cudaMemcpyAsync(&longest, tmp, sizeof(longest), cudaMemcpyDeviceToHost, st));
    TL_CUDA(cudaStreamSynchronize(st));
#undef TL_CUDA
    cleanup(false);
    ix.max_tok_list = longest;
    ix.tok_off = off;
    ix.tok_id = ids;
    ix.tok_doc = docs;
    return CHIMERA_OK;
}

// ------------------------------------------------------------------------------------------------ driver ---------
int build_index_device(Index &ix, const float *centroids, const int32_t *doclens, cudaStream_t st)
{
    int32_t *flags = nullptr;       // [0] validation bits, [1] max doc length
    int64_t *tmp = nullptr;
    int32_t *count = nullptr;
    auto cleanup = [&]() {
        cudaFree(flags);
        cudaFree(tmp);
        cudaFree(count);
    };
#define BUILD_CUDA(call)                                                                             \
    do {                                                                                             \
        cudaError_t e__ = (call);                                                                    \
        if (e__ != cudaSuccess) {                                                                    \
            cleanup();                                                                               \
            return fail(CHIMERA_CUDA_ERROR, "%s: %s", #call, cudaGetErrorString(e__));              \
        }                                                                                            \
    } while (0)

    const int64_t scan_n = ix.N > ix.K ? ix.N : ix.K;
    BUILD_CUDA(cudaMalloc(&flags, 2 * sizeof(int32_t)));
    BUILD_CUDA(cudaMalloc(&tmp, sizeof(int64_t) * ((scan_n + SCAN_TILE - 1) / SCAN_TILE + 1)));
    BUILD_CUDA(cudaMalloc(&count, sizeof(int32_t) * ix.K));
    BUILD_CUDA(cudaMemsetAsync(flags, 0, 2 * sizeof(int32_t), st));

    validate_kernel<<<ix.sm_count * 8, 256, 0, st>>>(ix.cids, ix.T, ix.K, doclens, ix.N, flags, flags + 1);
    BUILD_CUDA(cudaGetLastError());

    BUILD_CUDA(cudaMalloc(&ix.doc_off, sizeof(int64_t) * (ix.N + 1)));
    int rc = exclusive_scan(doclens, ix.N, ix.doc_off, tmp, st);
    if (rc) { cleanup(); return rc; }

    int32_t h_flags[2];
    int64_t total = 0;
    BUILD_CUDA(cudaMemcpyAsync(h_flags, flags, sizeof(h_flags), cudaMemcpyDeviceToHost, st));
    BUILD_CUDA(cudaMemcpyAsync(&total, ix.doc_off + ix.N, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    BUILD_CUDA(cudaStreamSynchronize(st));
    if (h_flags[0] & 1) { cleanup(); return fail(CHIMERA_INVALID_ARG, "a centroid id lies outside [0, n_centroids)"); }
    if (h_flags[0] & 2) { cleanup(); return fail(CHIMERA_INVALID_ARG, "a document length is < 1"); }
    if (total != ix.T) {
        cleanup();
        return fail(CHIMERA_INVALID_ARG, "document lengths sum to %lld, n_tokens is %lld", (long long)total,
                    (long long)ix.T);
    }
    ix.max_doclen = h_flags[1];

    // centroid digit planes
    BUILD_CUDA(cudaMalloc(&ix.cdig, (size_t)3 * ix.K * DIGIT_PITCH));
    BUILD_CUDA(cudaMemsetAsync(flags, 0, sizeof(int32_t), st));
    rc = launch_digits(centroids, ix.K, ix.D, ix.cdig, (uint32_t *)flags, st);
    if (rc) { cleanup(); return rc; }

    // inverted file
    BUILD_CUDA(cudaMemsetAsync(count, 0, sizeof(int32_t) * ix.K, st));
    int64_t warps_wanted = ix.N < (int64_t)ix.sm_count * 64 ? ix.N : (int64_t)ix.sm_count * 64;
    unsigned ivf_blocks = (unsigned)((warps_wanted * 32 + 255) / 256);
    ivf_kernel<0><<<ivf_blocks, 256, 0, st>>>(ix.cids, ix.doc_off, ix.N, count, nullptr, nullptr);
    BUILD_CUDA(cudaGetLastError());
    BUILD_CUDA(cudaMalloc(&ix.ivf_off, sizeof(int64_t) * (ix.K + 1)));
    rc = exclusive_scan(count, ix.K, ix.ivf_off, tmp, st);
    if (rc) { cleanup(); return rc; }
    BUILD_CUDA(cudaMemcpyAsync(&ix.ivf_len, ix.ivf_off + ix.K, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    BUILD_CUDA(cudaMemcpyAsync(h_flags, flags, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    BUILD_CUDA(cudaStreamSynchronize(st));
    if (h_flags[0] & ST_BAD_QUERY) { cleanup(); return fail(CHIMERA_INVALID_ARG, "a centroid element lies outside [-1, 1] or a centroid is longer than a unit vector"); }
    BUILD_CUDA(cudaMalloc(&ix.ivf_doc, sizeof(int32_t) * (size_t)(ix.ivf_len > 0 ? ix.ivf_len : 1)));
    BUILD_CUDA(cudaMemsetAsync(count, 0, sizeof(int32_t) * ix.K, st));
    ivf_kernel<1><<<ivf_blocks, 256, 0, st>>>(ix.cids, ix.doc_off, ix.N, count, ix.ivf_off, ix.ivf_doc);
    BUILD_CUDA(cudaGetLastError());
    BUILD_CUDA(cudaStreamSynchronize(st));
    cleanup();
#undef BUILD_CUDA
    return CHIMERA_OK;
}

}  // namespace chimera
