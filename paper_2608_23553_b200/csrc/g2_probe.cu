// Stage 2a: for each query token the nprobe centroids with the largest score (Sec. 3.2 step 1: the top-n_probe
// centroids of a query token), ordered by (score descending, centroid id ascending).
//
// The table is centroid-major [K][nq], so a warp reads one 128-byte row per step with lane = query token.  Every
// thread keeps a sorted list of its best P keys in shared memory (column layout list[j][thread], conflict-free); a
// key is a 64-bit integer whose order is (score desc, id asc).  Pass 1 turns slices of the table into partial lists,
// pass 2 folds the partial lists of a query into the final P per token.
#include <atomic>
#include <stdint.h>

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
// only_flagged: NULL, or int32[B]: blocks of queries whose entry is 0 return at once.
__global__ void __launch_bounds__(PROBE_THREADS)
probe_partial(const int32_t *__restrict__ table, int64_t K, int nq, int P, int rows_per_block, int n_part,
              unsigned long long *__restrict__ part, const int32_t *__restrict__ only_flagged)
{
    extern __shared__ unsigned long long lists[];    // [P][PROBE_THREADS]
    if (only_flagged && !only_flagged[blockIdx.y]) return;      // (fallback use: only the flagged queries)
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
probe_final(const unsigned long long *__restrict__ part, int nq, int P, int n_part, int32_t *__restrict__ probes,
            const int32_t *__restrict__ only_flagged)
{
    extern __shared__ unsigned long long lists[];      // [P][THREADS]
    if (only_flagged && !only_flagged[blockIdx.y]) return;
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
                              cudaStream_t st, const int32_t *only_flagged = nullptr)
{
    const dim3 grid(1, (unsigned)B, (unsigned)((nq + 31) / 32));
    const size_t per_thread = sizeof(unsigned long long) * (size_t)P;
    if (per_thread * 1024 <= 48 * 1024) {
        probe_final<1024><<<grid, 1024, per_thread * 1024, st>>>(part, nq, P, n_part, probes, only_flagged);
    } else if (per_thread * 512 <= 48 * 1024) {
        probe_final<512><<<grid, 512, per_thread * 512, st>>>(part, nq, P, n_part, probes, only_flagged);
    } else {
        const size_t smem = per_thread * PROBE_THREADS;
        if (smem > 48 * 1024)
            CHIMERA_CUDA(cudaFuncSetAttribute(probe_final<PROBE_THREADS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)smem));
        probe_final<PROBE_THREADS><<<grid, PROBE_THREADS, smem, st>>>(part, nq, P, n_part, probes, only_flagged);
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
    probe_partial<<<g1, PROBE_THREADS, smem, st>>>(table, ix.K, p.nq, p.P, rows_per_block, L.n_part, part, nullptr);
    CHIMERA_CUDA(cudaGetLastError());
    const int rc = launch_probe_final(part, p.B, p.nq, p.P, L.n_part, probes, st);
    if (rc) return rc;
    count_launch(SLOT_PROBE, 2);
    return CHIMERA_OK;
}

// =====================================================================================================================
// Probe side of stages 1 and 2a run together (launch_score_table_probes in g1_score_table.cu).
// =====================================================================================================================
constexpr int PQ_CAP = 1024;            // keys per queue: several times the expected number (see below)
constexpr int PQ_WARPS = 8;             // warps per block of the kernels below
constexpr int PQ_MAX_GROUPS = 256;      // groups of sample rows per query

int probe_queue_cap() { return PQ_CAP; }

// Every how-many-th centroid tile (128 centroids) is a sample tile, or 0 when the stages run separately.  The bound of
// a query-token row is (a little below) its nprobe-th best score among the sample, a fraction 1 / stride of the
// centroids, so about nprobe x stride centroids in all reach it (for exchangeable scores the count is
// negative-binomial with that mean); stride = 128 / max(nprobe, 4) keeps the mean near 128 keys, an eighth of PQ_CAP
// (for nprobe = 4 the chance of 1024 or more is below 1e-9 per row).  Strided tiles rather than the first ones, so
// that centroids stored in some spatial order still give a representative sample.
int probe_sample_stride(int64_t K, int nq, int P)
{
    if (P < 1 || P > 32 || nq < 1 || (nq & 3) != 0) return 0;
    const int stride = 128 / (P > 4 ? P : 4);              // 32, ..., 4
    const int64_t c_tiles = (K + 127) / 128;
    if (stride < 2 || c_tiles < 8 * (int64_t)stride) return 0;      // at least 8 sample tiles (1024 centroids)
    return stride;
}

int probe_queue_stride(const Index &ix, const Params &p) { return probe_sample_stride(ix.K, p.nq, p.P); }

// The sample rows of a query are cut into groups (16 rows or more, at most PQ_MAX_GROUPS groups, at least 64).
int probe_sample_groups(const Index &ix, int stride)
{
    const int64_t c_tiles = (ix.K + 127) / 128;
    const int64_t sample_rows = (c_tiles + stride - 1) / stride * 128;
    int64_t groups = sample_rows / 16;
    if (groups > PQ_MAX_GROUPS) groups = PQ_MAX_GROUPS;
    return (int)groups;
}

// Sample row r -> centroid: tile (r / 128) * stride, row r % 128 of it.
__device__ __forceinline__ int64_t sample_centroid(int64_t r, int stride) { return ((r >> 7) * stride << 7) + (r & 127); }

// grid (ceil(G / PQ_WARPS), B, ceil(nq / 32)): warp = one group of sample rows, lane = query token; the largest score
// of the group per token.  gmax: [B][G][nq].
__global__ void __launch_bounds__(32 * PQ_WARPS)
sample_max_kernel(const int32_t *__restrict__ table, int64_t K, int nq, int64_t sample_rows, int stride, int G,
                  int rows_per_group, int32_t *__restrict__ gmax)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = blockIdx.z * 32 + lane;
    const int b = blockIdx.y;
    const int g = blockIdx.x * PQ_WARPS + warp;
    if (g >= G || col >= nq) return;
    const int32_t *tb = table + (int64_t)b * K * nq + col;
    const int64_t r0 = (int64_t)g * rows_per_group;
    int64_t r1 = r0 + rows_per_group;
    if (r1 > sample_rows) r1 = sample_rows;
    int32_t best = INT32_MIN;
    for (int64_t r = r0; r < r1; r += 8) {
        int32_t v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int64_t c = sample_centroid(r + u, stride);
            v[u] = (r + u < r1 && c < K) ? tb[c * nq] : INT32_MIN;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) best = max(best, v[u]);
    }
    gmax[((int64_t)b * G + g) * nq + col] = best;
}

// One warp per query-token row: the nprobe-th largest of the row's G group maxima.  The nprobe largest maxima are
// nprobe different centroids, so the true nprobe-th best score is at least that: a bound.  Also empties the row's
// queue and clears the query's flag.
__global__ void __launch_bounds__(32 * PQ_WARPS)
sample_bound_kernel(const int32_t *__restrict__ gmax, int G, int nq, int P, int64_t rows, int32_t *__restrict__ thr,
                    int32_t *__restrict__ cnt, int32_t *__restrict__ ovf)
{
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * PQ_WARPS + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int64_t b = row / nq;
    const int col = (int)(row - b * nq);
    // (value, group) keys are distinct, so "the largest key below the previous one" walks down the order
    unsigned long long mine[PQ_MAX_GROUPS / 32];
#pragma unroll
    for (int i = 0; i < PQ_MAX_GROUPS / 32; ++i) {
        const int g = lane + 32 * i;
        mine[i] = g < G ? key_int(gmax[(b * G + g) * nq + col], g) : 0ull;
    }
    unsigned long long prev = ~0ull;
    for (int j = 0; j < P; ++j) {
        unsigned long long best = 0ull;
#pragma unroll
        for (int i = 0; i < PQ_MAX_GROUPS / 32; ++i)
            if (mine[i] < prev && mine[i] > best) best = mine[i];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            if (other > best) best = other;
        }
        prev = best;
    }
    if (lane == 0) {
        thr[row] = (int32_t)((uint32_t)(prev >> 32) ^ 0x80000000u);
        cnt[row] = 0;
        if (col == 0) ovf[b] = 0;
    }
}

// Same grid as sample_max_kernel: the sample rows once more, every score at or above the row's bound into its queue
// (the rest of the table does this in the score-table kernel's epilogue).
__global__ void __launch_bounds__(32 * PQ_WARPS)
sample_push_kernel(const int32_t *__restrict__ table, int64_t K, int nq, int64_t sample_rows, int stride, int G,
                   int rows_per_group, const int32_t *__restrict__ thr, int32_t *__restrict__ cnt,
                   unsigned long long *__restrict__ keys, int cap)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = blockIdx.z * 32 + lane;
    const int b = blockIdx.y;
    const int g = blockIdx.x * PQ_WARPS + warp;
    if (g >= G || col >= nq) return;
    const int32_t *tb = table + (int64_t)b * K * nq + col;
    const int64_t row = (int64_t)b * nq + col;
    const int32_t bound = thr[row];
    const int64_t r0 = (int64_t)g * rows_per_group;
    int64_t r1 = r0 + rows_per_group;
    if (r1 > sample_rows) r1 = sample_rows;
    for (int64_t r = r0; r < r1; r += 8) {
        int32_t v[8];
        int64_t c[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            c[u] = sample_centroid(r + u, stride);
            v[u] = (r + u < r1 && c[u] < K) ? tb[c[u] * nq] : INT32_MIN;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (v[u] >= bound && r + u < r1 && c[u] < K) {
                const int slot = atomicAdd(cnt + row, 1);
                if (slot < cap) keys[row * cap + slot] = key_int(v[u], (int32_t)c[u]);
            }
        }
    }
}

// One warp per query-token row: the nprobe best keys of the row's queue -> probes[row].  A row whose queue
// overflowed flags its query instead.
__global__ void __launch_bounds__(32 * PQ_WARPS)
probe_merge_kernel(int nq, int P, int64_t rows, const int32_t *__restrict__ cnt,
                   const unsigned long long *__restrict__ keys, int cap, int32_t *__restrict__ probes,
                   int32_t *__restrict__ ovf)
{
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * PQ_WARPS + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int n = cnt[row];
    if (n > cap) {
        if (lane == 0) ovf[row / nq] = 1;
        return;
    }
    const unsigned long long *mine = keys + row * cap;
    unsigned long long prev = ~0ull;
    int32_t my_id = 0;
    for (int j = 0; j < P; ++j) {                            // keys are distinct (they contain the centroid id)
        unsigned long long best = 0ull;
        for (int i = lane; i < n; i += 32) {
            const unsigned long long k = __ldg(mine + i);
            if (k < prev && k > best) best = k;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            if (other > best) best = other;
        }
        prev = best;
        if (lane == j) my_id = key_id(best);
    }
    if (lane < P) probes[row * P + lane] = my_id;            // (the queue holds at least nprobe keys: the group maxima)
}

int launch_probe_sample(const Index &ix, const Params &p, const Layout &L, const int32_t *table, char *ws,
                        int n_sample_tiles, cudaStream_t st)
{
    const int64_t sample_rows = (int64_t)n_sample_tiles * 128;
    const int G = L.pq_groups;
    const int rows_per_group = (int)((sample_rows + G - 1) / G);
    const int64_t rows = (int64_t)p.B * p.nq;
    int32_t *gmax = (int32_t *)(ws + L.pq_gmax), *thr = (int32_t *)(ws + L.pq_thr), *cnt = (int32_t *)(ws + L.pq_cnt);
    int32_t *ovf = (int32_t *)(ws + L.pq_ovf);
    unsigned long long *keys = (unsigned long long *)(ws + L.pq_keys);
    const dim3 grid((unsigned)((G + PQ_WARPS - 1) / PQ_WARPS), (unsigned)p.B, (unsigned)((p.nq + 31) / 32));
    sample_max_kernel<<<grid, 32 * PQ_WARPS, 0, st>>>(table, ix.K, p.nq, sample_rows, L.pq_stride, G, rows_per_group,
                                                      gmax);
    CHIMERA_CUDA(cudaGetLastError());
    sample_bound_kernel<<<(unsigned)((rows + PQ_WARPS - 1) / PQ_WARPS), 32 * PQ_WARPS, 0, st>>>(gmax, G, p.nq, p.P, rows,
                                                                                                thr, cnt, ovf);
    CHIMERA_CUDA(cudaGetLastError());
    sample_push_kernel<<<grid, 32 * PQ_WARPS, 0, st>>>(table, ix.K, p.nq, sample_rows, L.pq_stride, G, rows_per_group,
                                                       thr, cnt, keys, L.pq_cap);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_PROBE, 3);
    return CHIMERA_OK;
}

int launch_probe_merge(const Index &ix, const Params &p, const Layout &L, const int32_t *table, char *ws, cudaStream_t st)
{
    const int64_t rows = (int64_t)p.B * p.nq;
    const int32_t *cnt = (const int32_t *)(ws + L.pq_cnt);
    const unsigned long long *keys = (const unsigned long long *)(ws + L.pq_keys);
    int32_t *ovf = (int32_t *)(ws + L.pq_ovf);
    unsigned long long *part = (unsigned long long *)(ws + L.part);
    int32_t *probes = (int32_t *)(ws + L.probes);
    probe_merge_kernel<<<(unsigned)((rows + PQ_WARPS - 1) / PQ_WARPS), 32 * PQ_WARPS, 0, st>>>(p.nq, p.P, rows, cnt, keys,
                                                                                               L.pq_cap, probes, ovf);
    CHIMERA_CUDA(cudaGetLastError());
    // queries with an overflowed queue (none, except for inputs with masses of equal scores): the table scan, whose
    // blocks return at once for every other query
    const size_t smem = sizeof(unsigned long long) * (size_t)p.P * PROBE_THREADS;
    if (smem > 48 * 1024)
        CHIMERA_CUDA(cudaFuncSetAttribute(probe_partial, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int rows_per_block = (int)((ix.K + L.probe_blocks - 1) / L.probe_blocks);
    const unsigned col_groups = (unsigned)((p.nq + 31) / 32);
    probe_partial<<<dim3((unsigned)L.probe_blocks, (unsigned)p.B, col_groups), PROBE_THREADS, smem, st>>>(
        table, ix.K, p.nq, p.P, rows_per_block, L.n_part, part, ovf);
    CHIMERA_CUDA(cudaGetLastError());
    const int rc = launch_probe_final(part, p.B, p.nq, p.P, L.n_part, probes, st, ovf);
    if (rc) return rc;
    count_launch(SLOT_PROBE, 3);
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

extern "C" int32_t chimera_probe_sample_stride(int64_t n_centroids, int32_t q_len, int32_t nprobe)
{
    return chimera::probe_sample_stride(n_centroids, q_len, nprobe);
}

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
        score_table, n_centroids, q_len, nprobe, rows_per_block, n_part, part, nullptr);
    CHIMERA_CUDA(cudaGetLastError());
    return launch_probe_final(part, n_queries, q_len, nprobe, n_part, out_probes, st);
}
