// KV gather / compaction (Section 3.1, X[Id]; Section 3.3, KV_cache[Id_sink, Id_entropy]):
// dst[p][j][:] = src[p][keep[j]][:] for every K and V plane, all planes in one launch.
//
// Pure data movement, bound by HBM bandwidth (each moved row is read once and written
// once).  A "worker" is one warp that owns a ring of shared-memory stages and walks the
// moved rows of one plane front to back, 32 rows (one chunk) at a time:
//   - the lanes issue TMA bulk loads global -> shared, one per run of consecutive source
//     rows, completing on the stage's mbarrier;
//   - a few chunks later lane 0 waits for that mbarrier and issues ONE bulk store
//     shared -> global for the whole chunk (destination rows are contiguous).
// In place (dst == src) this order is race free: the keep list is strictly ascending with
// keep[j] >= j, so a chunk's sources lie at or behind its own first destination row.
// A chunk is stored only after its loads and those of all earlier chunks have landed,
// and later chunks only read rows behind everything stored so far.  Planes are
// independent, so the ring keeps streaming across plane boundaries.
#include "common.cuh"

namespace sirllm {

namespace {

constexpr int kChunkRows = 32;    // rows per chunk = one per lane
constexpr int kStoreSlack = 2;    // bulk stores that may still be reading shared memory
constexpr int kMaxStages = 12;
constexpr uint32_t kSpinLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes,
                                          uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
            "r"(smem_u32(smem_dst)),
        "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
                 "r"(smem_u32(smem_src)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() {
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

struct WorkerRing {
    uint64_t* full;      // [stages] mbarriers
    char** st_dst;       // [stages] destination of the chunk held by the stage
    uint32_t* st_bytes;  // [stages]
    char* buf;           // stages * stage_bytes
};

// Lane 0 waits for the loads of chunk c and stores it.  Returns false on timeout.
__device__ __forceinline__ bool store_chunk(const WorkerRing& ring, int64_t c, int stages,
                                            uint32_t stage_bytes, int lane) {
    bool ok = true;
    if (lane == 0) {
        const int stage = (int)(c % stages);
        const uint32_t parity = (uint32_t)((c / stages) & 1);
        uint32_t spins = 0;
        while (!mbar_try_wait(&ring.full[stage], parity)) {
            if (++spins > kSpinLimit) {
                ok = false;
                break;
            }
        }
        if (ok) {
            bulk_store(ring.st_dst[stage], ring.buf + (size_t)stage * stage_bytes,
                       ring.st_bytes[stage]);
            bulk_commit();
        }
    }
    return __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
}

__global__ void __launch_bounds__(256, 1)
compact_kernel(const CompactParams p, const int stages, const int n_units) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int n_workers = blockDim.x >> 5;
    const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t stage_bytes = (uint32_t)kChunkRows * (uint32_t)p.row_bytes;

    // shared memory: [workers][stages] mbarriers, destinations, sizes; then the rings
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw);
    char** dsts = reinterpret_cast<char**>(bars + n_workers * kMaxStages);
    uint32_t* sizes = reinterpret_cast<uint32_t*>(dsts + n_workers * kMaxStages);
    size_t header = (size_t)n_workers * kMaxStages * (8 + 8 + 4);
    header = (header + 127) & ~(size_t)127;
    WorkerRing ring;
    ring.full = bars + wid * kMaxStages;
    ring.st_dst = dsts + wid * kMaxStages;
    ring.st_bytes = sizes + wid * kMaxStages;
    ring.buf = reinterpret_cast<char*>(smem_raw) + header + (size_t)wid * stages * stage_bytes;

    if (lane == 0) {
        for (int i = 0; i < stages; ++i) mbar_init(&ring.full[i], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    grid_dependency_wait();  // the keep lists of the selection kernel

    const int lead = stages - 1 - kStoreSlack;  // chunks whose loads run ahead of the stores
    const int64_t g = (int64_t)blockIdx.x * n_workers + wid;
    const int64_t G = (int64_t)gridDim.x * n_workers;
    int64_t it = 0;      // chunks whose loads were issued
    int64_t stored = 0;  // chunks whose store was issued
    bool alive = true;

    for (int64_t u = g; u < n_units && alive; u += G) {
        const int tensor = (int)(u / p.planes_per_tensor);
        const int64_t plane = u - (int64_t)tensor * p.planes_per_tensor;
        const int s = (int)(plane / p.planes_per_stream);
        const int n = min(max(p.n_keep[s], 0), p.keep_stride);
        int f = p.first_moved[s];
        if (f < 0) continue;  // keep list rejected
        if (!p.in_place) f = 0;
        const char* src = (tensor ? p.src[1] : p.src[0]) + (size_t)plane * p.capacity * p.row_bytes;
        char* dst = (tensor ? p.dst[1] : p.dst[0]) + (size_t)plane * p.capacity * p.row_bytes;
        const int32_t* keep = p.keep_idx + (size_t)s * p.keep_stride;

        int kj_next = f + lane < n ? keep[f + lane] : -2;  // source rows of the first chunk
        for (int j0 = f; j0 < n && alive; j0 += kChunkRows) {
            const int nrows = min(kChunkRows, n - j0);
            const int stage = (int)(it % stages);
            const int kj = kj_next;
            // fetch the next chunk's source rows now; they are needed one trip later
            kj_next = j0 + kChunkRows + lane < n ? keep[j0 + kChunkRows + lane] : -2;
            if (lane == 0) {
                if (it >= stages) bulk_wait_read<kStoreSlack>();  // the stage's last store has left
                ring.st_dst[stage] = dst + (size_t)j0 * p.row_bytes;
                ring.st_bytes[stage] = (uint32_t)nrows * p.row_bytes;
                mbar_expect_tx(&ring.full[stage], (uint32_t)nrows * p.row_bytes);
            }
            __syncwarp();
            // one bulk load per run of consecutive source rows
            const int prev = __shfl_up_sync(0xFFFFFFFFu, kj, 1);
            const bool head = lane < nrows && (lane == 0 || kj != prev + 1);
            const uint32_t heads = __ballot_sync(0xFFFFFFFFu, head);
            if (head) {
                const uint32_t later = lane == 31 ? 0u : (heads & ~((2u << lane) - 1u));
                const int next = later ? __ffs(later) - 1 : nrows;
                bulk_load(ring.buf + (size_t)stage * stage_bytes + (size_t)lane * p.row_bytes,
                          src + (size_t)kj * p.row_bytes, (uint32_t)(next - lane) * p.row_bytes,
                          &ring.full[stage]);
            }
            ++it;
            if (it - stored > lead) {
                alive = store_chunk(ring, stored, stages, stage_bytes, lane);
                ++stored;
            }
        }
    }
    while (alive && stored < it) {
        alive = store_chunk(ring, stored, stages, stage_bytes, lane);
        ++stored;
    }
    if (lane == 0) {
        if (!alive) atomicOr(p.status, SIRLLM_STATUS_TIMEOUT);
        bulk_wait_all();
    }
}

// Checks caller-supplied keep lists and finds, per stream, the first slot whose row moves.
__global__ void compact_plan_kernel(const CompactParams p, int32_t* __restrict__ first_moved) {
    __shared__ int sh_first, sh_bad;
    const int s = blockIdx.x;
    const int n = min(max(p.n_keep[s], 0), p.keep_stride);
    const int32_t* keep = p.keep_idx + (size_t)s * p.keep_stride;
    if (threadIdx.x == 0) {
        sh_first = n;
        sh_bad = (p.n_keep[s] < 0 || p.n_keep[s] > p.keep_stride) ? 1 : 0;
    }
    __syncthreads();
    for (int j = threadIdx.x; j < n; j += blockDim.x) {
        const int kj = keep[j];
        const int prev = j > 0 ? keep[j - 1] : -1;
        if (kj <= prev || kj >= p.capacity) sh_bad = 1;
        if (kj != j) atomicMin(&sh_first, j);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (sh_bad) {
            atomicOr(p.status, SIRLLM_STATUS_BAD_KEEP);
            first_moved[s] = -1;
        } else {
            first_moved[s] = sh_first;
        }
    }
}

}  // namespace

cudaError_t launch_compact_plan(const CompactParams& p, int n_streams, int32_t* first_moved,
                                cudaStream_t st) {
    compact_plan_kernel<<<n_streams, 256, 0, st>>>(p, first_moved);
    return cudaGetLastError();
}

cudaError_t launch_compact(const CompactParams& p, cudaStream_t st, bool overlap) {
    int n_tensors = 0;
    CompactParams q = p;
    for (int t = 0; t < 2; ++t) {
        if (p.src[t] != nullptr) {
            q.src[n_tensors] = p.src[t];
            q.dst[n_tensors] = p.dst[t];
            ++n_tensors;
        }
    }
    const int64_t units64 = (int64_t)n_tensors * p.planes_per_tensor;
    if (units64 == 0) return cudaSuccess;
    if (units64 > 0x7FFFFFFF) return cudaErrorInvalidValue;
    const int n_units = (int)units64;

    int dev = 0, n_sm = 0, smem_max = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) return e;

    // ring geometry: as many workers per SM as fit with at least 6 stages each (at most 8)
    const size_t stage_bytes = (size_t)kChunkRows * p.row_bytes;
    const size_t budget = (size_t)smem_max - 1024;
    int workers = 4, stages = 6;
    while (workers > 1 && (size_t)workers * stages * stage_bytes > budget) --workers;
    while (stages > 4 && (size_t)workers * stages * stage_bytes > budget) --stages;
    if ((size_t)workers * stages * stage_bytes > budget) return cudaErrorInvalidValue;
    while (stages < 8 && (size_t)workers * (stages + 1) * stage_bytes <= budget) ++stages;
    size_t header = (size_t)workers * kMaxStages * (8 + 8 + 4);
    header = (header + 127) & ~(size_t)127;
    const size_t smem = header + (size_t)workers * stages * stage_bytes;
    e = cudaFuncSetAttribute(compact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int grid = (int)((n_units + workers - 1) / workers < n_sm ? (n_units + workers - 1) / workers
                                                                    : n_sm);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)workers * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, compact_kernel, q, stages, n_units);
}

}  // namespace sirllm
