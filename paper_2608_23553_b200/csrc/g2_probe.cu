// Stage 2a: for each query token the nprobe centroids with the largest score (Sec. 3.2 step 1: the top-n_probe
// centroids of a query token), ordered by (score descending, centroid id ascending).
//
// The table is centroid-major [K][nq], so a warp reads one 128-byte row per step with lane = query token.  Every
// thread keeps a sorted list of its best P keys in shared memory (column layout list[j][thread], conflict-free); a
// key is a 64-bit integer whose order is (score desc, id asc).  Pass 1 turns slices of the table into partial lists,
// pass 2 folds the partial lists of a query into the final P per token.
#include <atomic>

#include "common.cuh"

namespace chimera {

constexpr int PROBE_THREADS = PROBE_WARPS * 32;

template <int STRIDE = PROBE_THREADS>
__device__ __forceinline__ void list_insert(unsigned long long *list, int P, unsigned long long key)
{
    // list[j * STRIDE] is entry j of this thread's list, descending.
    if (key <= list[(P - 1) * STRIDE]) return;
    int j = P - 1;
    while (j > 0) {
        unsigned long long up = list[(j - 1) * STRIDE];
        if (up >= key) break;
        list[j * STRIDE] = up;
        --j;
    }
    list[j * STRIDE] = key;
}

// grid (probe_blocks, B, ceil(nq / 32)).  part: [B][n_part][P][nq], n_part = probe_blocks (one list per block).
__global__ void __launch_bounds__(PROBE_THREADS)
probe_partial(const int32_t *__restrict__ table, int64_t K, int nq, int P, int rows_per_block, int n_part,
              unsigned long long *__restrict__ part)
{
    extern __shared__ unsigned long long lists[];    // [P][PROBE_THREADS]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = blockIdx.z * 32 + lane;
    const int b = blockIdx.y;
    unsigned long long *mine = lists + threadIdx.x;
    for (int j = 0; j < P; ++j) mine[j * PROBE_THREADS] = 0ull;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_block;
    int64_t r1 = r0 + rows_per_block;
    if (r1 > K) r1 = K;
    if (col < nq) {
        const int32_t *tb = table + (int64_t)b * K * nq + col;
        int64_t r = r0 + warp;
        // sixteen independent loads in flight per thread (the stream is bound by bytes in flight)
        for (; r + 15 * PROBE_WARPS < r1; r += 16 * PROBE_WARPS) {
            int32_t sc[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) sc[u] = tb[(r + u * PROBE_WARPS) * nq];
#pragma unroll
            for (int u = 0; u < 16; ++u) list_insert(mine, P, key_int(sc[u], (int32_t)(r + u * PROBE_WARPS)));
        }
        for (; r < r1; r += PROBE_WARPS) list_insert(mine, P, key_int(tb[r * nq], (int32_t)r));
    }
    // fold the block's eight lists into warp 0's, then write one list per block and column
    __syncthreads();
    if (warp == 0 && col < nq) {
        for (int w = 1; w < PROBE_WARPS; ++w) {
            const unsigned long long *src = lists + w * 32 + lane;
            for (int j = 0; j < P; ++j) {
                unsigned long long key = src[j * PROBE_THREADS];
                if (key <= mine[(P - 1) * PROBE_THREADS]) break;
                list_insert(mine, P, key);
            }
        }
        unsigned long long *dst = part + (((int64_t)b * n_part + blockIdx.x) * P) * nq + col;
        for (int j = 0; j < P; ++j) dst[(int64_t)j * nq] = mine[j * PROBE_THREADS];
    }
}

// grid (1, B, ceil(nq / 32)), THREADS threads.  Folds n_part sorted lists per column into one; writes
// probes[b][col][0..P).  Warp w takes lists w, w + W, ... (W = THREADS / 32 warps, lane = column); the warps' lists are
// then folded pairwise in a tree.  With one query per call this kernel is a single block, so it is latency that counts:
// up to eight list heads are loaded together, and 32 warps share the lists when nprobe is small enough for the
// shared-memory lists of 1024 threads.
template <int THREADS>
__global__ void __launch_bounds__(THREADS)
probe_final(const unsigned long long *__restrict__ part, int nq, int P, int n_part, int32_t *__restrict__ probes)
{
    extern __shared__ unsigned long long lists[];      // [P][THREADS]
    constexpr int W = THREADS / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = blockIdx.z * 32 + lane;
    const int b = blockIdx.y;
    unsigned long long *mine = lists + threadIdx.x;
    for (int j = 0; j < P; ++j) mine[j * THREADS] = 0ull;
    if (col < nq) {
        if (P <= 4 && n_part <= 8 * W) {
            // Few lists per warp (one query per call): walking a list key by key is a chain of dependent loads, and
            // with an empty running list every key of every list qualifies anyway -- so all keys of four lists are
            // loaded together (16 independent loads), twice.
            for (int l0 = warp; l0 < n_part; l0 += 4 * W) {
                unsigned long long k[4][4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int l = l0 + u * W;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        k[u][j] = (l < n_part && j < P) ? part[((((int64_t)b * n_part + l) * P) + j) * nq + col] : 0ull;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (k[u][j] > mine[(P - 1) * THREADS]) list_insert<THREADS>(mine, P, k[u][j]);
            }
        } else {
            // a list is only walked further while its keys still beat this thread's current P-th best
            for (int l0 = warp; l0 < n_part; l0 += 8 * W) {
                unsigned long long head[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int l = l0 + u * W;
                    head[u] = l < n_part ? part[(((int64_t)b * n_part + l) * P) * nq + col] : 0ull;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int l = l0 + u * W;
                    if (l >= n_part || head[u] <= mine[(P - 1) * THREADS]) continue;
                    list_insert<THREADS>(mine, P, head[u]);
                    const unsigned long long *src = part + (((int64_t)b * n_part + l) * P) * nq + col;
                    for (int j = 1; j < P; ++j) {
                        unsigned long long key = src[(int64_t)j * nq];
                        if (key <= mine[(P - 1) * THREADS]) break;      // source list is descending
                        list_insert<THREADS>(mine, P, key);
                    }
                }
            }
        }
    }
    for (int s = W / 2; s >= 1; s >>= 1) {
        __syncthreads();
        if (warp < s && col < nq) {
            const unsigned long long *src = lists + (warp + s) * 32 + lane;
            for (int j = 0; j < P; ++j) {
                unsigned long long key = src[j * THREADS];
                if (key <= mine[(P - 1) * THREADS]) break;
                list_insert<THREADS>(mine, P, key);
            }
        }
    }
    if (warp == 0 && col < nq) {
        int32_t *dst = probes + ((int64_t)b * nq + col) * P;
        for (int j = 0; j < P; ++j) dst[j] = key_id(mine[j * THREADS]);
    }
}

// The widest block whose lists (nprobe keys of 8 bytes per thread) fit the default 48 KB of shared memory, at least
// PROBE_THREADS (whose lists may need the opt-in limit: 128 KB at nprobe = 64).
static int launch_probe_final(const unsigned long long *part, int B, int nq, int P, int n_part, int32_t *probes,
                              cudaStream_t st)
{
    const dim3 grid(1, (unsigned)B, (unsigned)((nq + 31) / 32));
    const size_t per_thread = sizeof(unsigned long long) * (size_t)P;
    if (per_thread * 1024 <= 48 * 1024) {
        probe_final<1024><<<grid, 1024, per_thread * 1024, st>>>(part, nq, P, n_part, probes);
    } else if (per_thread * 512 <= 48 * 1024) {
        probe_final<512><<<grid, 512, per_thread * 512, st>>>(part, nq, P, n_part, probes);
    } else {
        const size_t smem = per_thread * PROBE_THREADS;
        if (smem > 48 * 1024)
            CHIMERA_CUDA(cudaFuncSetAttribute(probe_final<PROBE_THREADS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)smem));
        probe_final<PROBE_THREADS><<<grid, PROBE_THREADS, smem, st>>>(part, nq, P, n_part, probes);
    }
    CHIMERA_CUDA(cudaGetLastError());
    return CHIMERA_OK;
}

int launch_probes(const Index &ix, const Params &p, const Layout &L, const int32_t *table, unsigned long long *part,
                  int32_t *probes, cudaStream_t st)
{
    const size_t smem = sizeof(unsigned long long) * (size_t)p.P * PROBE_THREADS;
    if (smem > 48 * 1024)
        CHIMERA_CUDA(cudaFuncSetAttribute(probe_partial, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int rows_per_block = (int)((ix.K + L.probe_blocks - 1) / L.probe_blocks);
    const unsigned col_groups = (unsigned)((p.nq + 31) / 32);
    dim3 g1((unsigned)L.probe_blocks, (unsigned)p.B, col_groups);
    probe_partial<<<g1, PROBE_THREADS, smem, st>>>(table, ix.K, p.nq, p.P, rows_per_block, L.n_part, part);
    CHIMERA_CUDA(cudaGetLastError());
    const int rc = launch_probe_final(part, p.B, p.nq, p.P, L.n_part, probes, st);
    if (rc) return rc;
    count_launch(SLOT_PROBE, 2);
    return CHIMERA_OK;
}

// =====================================================================================================================
// Allocation-free variant of the probe stage.
//
// Some callers cannot allocate device memory at all: latency-critical serving loops that size everything at start-up
// and forbid allocator calls afterwards (an allocation can synchronise the device or fail late), and processes in
// which another component owns the device memory pool, so that a cudaMalloc from here would fail or take memory that
// was promised elsewhere.  For them this entry point runs the same two kernels as the probe stage but keeps the partial
// lists (the stage's only scratch) in a fixed array that is part of the library image: nothing is allocated or freed
// and no workspace is passed.
//
// The array below lives on every GPU that loads the library, from load until the process exits.  All calls share it
// and it keeps the last call's contents.
// =====================================================================================================================
constexpr size_t STATIC_PROBE_SCRATCH_BYTES = 4u << 20;     // 4 MiB
static __device__ __align__(256) unsigned long long g_probe_scratch[STATIC_PROBE_SCRATCH_BYTES / 8];

constexpr int STATIC_MAX_DEVICES = 64;
// Device address of g_probe_scratch on each device (0 = not looked up yet).  In host code the symbol's name is only a
// handle for the runtime, not a device address: it must be translated with cudaGetSymbolAddress, with the device in
// question current, before a kernel can be given it.
// Host threads may make their first calls at the same time: the entries are atomics (every writer stores the same
// address, so relaxed ordering is enough).  A cached address does not survive cudaDeviceReset.
static std::atomic<unsigned long long *> g_probe_scratch_ptr[STATIC_MAX_DEVICES];

}  // namespace chimera

extern "C" int chimera_probes_static(const int32_t *score_table, int64_t n_centroids, int32_t n_queries, int32_t q_len,
                                     int32_t nprobe, void *stream, int32_t *out_probes)
{
    using namespace chimera;
    if (!score_table || !out_probes) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    if (n_centroids < 1 || n_centroids > 0x7fffffffLL) return fail(CHIMERA_INVALID_ARG, "n_centroids out of range");
    if (n_queries < 1 || n_queries > 65535) return fail(CHIMERA_INVALID_ARG, "n_queries must be in [1, 65535]");
    if (q_len < 1 || q_len > CHIMERA_MAX_QLEN) return fail(CHIMERA_INVALID_ARG, "q_len must be in [1, %d]", CHIMERA_MAX_QLEN);
    if (nprobe < 1 || nprobe > CHIMERA_MAX_NPROBE || nprobe > n_centroids)
        return fail(CHIMERA_INVALID_ARG, "nprobe must be in [1, min(n_centroids, %d)]", CHIMERA_MAX_NPROBE);

    int dev = 0, sm_count = 0;
    CHIMERA_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return fail(CHIMERA_UNSUPPORTED, "device ordinal %d is not supported", dev);
    CHIMERA_CUDA(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
    unsigned long long *part = g_probe_scratch_ptr[dev].load(std::memory_order_relaxed);
    if (!part) {                              // first call on this device (it is the current one)
        void *p = nullptr;
        CHIMERA_CUDA(cudaGetSymbolAddress(&p, g_probe_scratch));
        part = static_cast<unsigned long long *>(p);
        g_probe_scratch_ptr[dev].store(part, std::memory_order_relaxed);
    }

    // same slicing rule as the workspace-based stage: about four blocks per SM over the batch, at most 512 per query,
    // at least ~256 rows per block; one partial list per block
    int64_t blocks = (4LL * sm_count + n_queries - 1) / n_queries;
    const int64_t by_rows = (n_centroids + 255) / 256;
    if (blocks > by_rows) blocks = by_rows;
    if (blocks > 512) blocks = 512;
    if (blocks < 1) blocks = 1;
    const int n_part = (int)blocks;
    const size_t need = sizeof(unsigned long long) * (size_t)n_queries * n_part * nprobe * q_len;
    if (need > STATIC_PROBE_SCRATCH_BYTES)
        return fail(CHIMERA_WORKSPACE_TOO_SMALL,
                    "this call needs %zu bytes of probe scratch; the built-in array holds %zu (use chimera_search with "
                    "a workspace for larger problems)", need, (size_t)STATIC_PROBE_SCRATCH_BYTES);

    cudaStream_t st = (cudaStream_t)stream;
    const size_t smem = sizeof(unsigned long long) * (size_t)nprobe * PROBE_THREADS;
    if (smem > 48 * 1024)
        CHIMERA_CUDA(cudaFuncSetAttribute(probe_partial, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int rows_per_block = (int)((n_centroids + blocks - 1) / blocks);
    const unsigned col_groups = (unsigned)((q_len + 31) / 32);
    // probe_partial writes every entry probe_final reads (all n_part lists x nprobe keys x q_len columns), so nothing
    // of the previous call's contents survives into this call's result and nothing needs clearing.
    probe_partial<<<dim3((unsigned)blocks, (unsigned)n_queries, col_groups), PROBE_THREADS, smem, st>>>(
        score_table, n_centroids, q_len, nprobe, rows_per_block, n_part, part);
    CHIMERA_CUDA(cudaGetLastError());
    return launch_probe_final(part, n_queries, q_len, nprobe, n_part, out_probes, st);
}
