// KV gather / compaction (Section 3.1, X[Id]; Section 3.3, KV_cache[Id_sink, Id_entropy]):
// dst[p][j][:] = src[p][keep[j]][:] for every K and V plane, all planes in one launch.
//
// Pure data movement, bound by HBM bandwidth (each moved row is read once and written
// once).  A "worker" is one warp that owns a ring of shared-memory stages and walks a run
// of moved rows of one plane front to back, 32 rows (one chunk) at a time:
//   - the lanes issue TMA bulk loads global -> shared, one per run of consecutive source
//     rows, completing on the stage's mbarrier;
//   - a few chunks later lane 0 waits for that mbarrier and issues ONE bulk store
//     shared -> global for the whole chunk (destination rows are contiguous).
// The ring keeps streaming across the boundaries of the worker's work units.
//
// In place (dst == src) this order is race free: the keep list is strictly ascending with
// keep[j] >= j, so a chunk's sources lie at or behind its own first destination row.  A
// chunk is stored only after its loads and those of all earlier chunks of the plane have
// landed, and later chunks only read rows behind everything stored so far.
//
// To fill all SMs evenly, the moved rows of a plane are cut into segments of `seg_chunks` chunks that
// different workers take.  Work units (plane, segment) are numbered segment-major, so a
// plane's earlier segments come long before its later ones, and are handed out in that order
// through one ticket counter in the workspace: a worker that is about to run dry draws the
// next number.  That evens out SMs that run at different speeds.
//
// A segment's stores overwrite rows that may still be the sources of EARLIER segments of the
// plane (never of later ones: keep[j] >= j).  Every segment therefore publishes how many of
// its chunks have landed in shared memory (one 64-bit progress word per plane and segment:
// compaction epoch | chunk count).  Before a chunk with destination
// rows [d0, d1) is stored, the worker makes sure that every destination row j in front of
// its segment whose source keep[j] lies below d1 has landed: it reads the earlier segments'
// progress words (one per lane, acquire), finds J = the number of leading rows of the plane
// known to have landed, and may then store anything below keep[J] (all of the plane once the
// earlier segments are complete).  The bound is remembered, so a segment polls again only
// when it outruns it; with rows moving by many slots, the rows a segment overwrites were read
// long before.  The wait has an iteration limit.  A worker only ever waits for units with a
// smaller number than its own, and every smaller number was drawn by a worker that is
// running (it drew the number itself), so by induction the waits end whatever number of CTAs
// the device keeps resident at once.
#include <atomic>

#include "common.cuh"

namespace sirllm {

namespace {

constexpr int kChunkRows = 32;  // rows per chunk = one per lane
constexpr int kStoreSlack = 1;  // bulk stores that may still be reading shared memory
constexpr int kMaxStages = 8;
constexpr int kIdxAhead = 4;     // chunks whose source indices are fetched ahead
constexpr int kMaxWorkers = 4;   // worker warps per CTA
constexpr int kPublishEvery = 4; // chunks between two updates of a segment's progress word
constexpr int kNoBound = 0x7FFFFFFF;
constexpr int kUnitsPerWorker = 16;  // work units per worker the split of the planes aims at
constexpr int kMinSegChunks = 5;     // shortest segment (chunks) worth a unit's set-up
constexpr int64_t kSmallJobBytes = 8 << 20;  // planes x longest keep list x row: the two-phase kernel's range

// What the store of a chunk needs to know about the chunk ...
struct StageInfo {
    char* dst;         // destination of the chunk held by the stage
    uint32_t bytes;
    int32_t d_end;     // one past the chunk's last destination row; 0: no earlier segment to mind
    uint32_t publish;  // != 0: chunks of this segment that have landed once this one has
    uint32_t unit;     // running number of the worker's work unit the chunk belongs to
};
// ... and about the work unit (plane, segment) it belongs to; written once per unit.
struct UnitInfo {
    const int32_t* keep;       // keep list of the unit's stream
    unsigned long long* prog;  // progress words of the unit's plane, one per segment
    int32_t seg;               // segment of the plane
    int32_t first;             // first moved row of the stream
    int32_t seg_rows;          // rows per (full) segment
    int32_t n;                 // rows kept in the stream
};

// What a worker knows about the earlier segments of the unit it is storing.
struct SafeBound {
    uint32_t unit = 0xFFFFFFFFu;
    int32_t below = 0;  // destination rows below this one may be stored
};

// Before a chunk of a later segment is stored: wait (whole warp, at most `limit` polls) until
// no earlier segment of the plane still has to read the rows below d_end.
__device__ __forceinline__ bool wait_for_earlier_segments(const UnitInfo& ui, int32_t d_end, uint32_t unit,
                                                          uint32_t epoch, SafeBound& safe, int lane,
                                                          uint32_t limit) {
    if (safe.unit != unit) {
        safe.unit = unit;
        safe.below = 0;
    }
    uint32_t polls = 0;
    while (d_end > safe.below) {
        // lane g looks at segment g < seg: has it landed all its chunks, if not how many
        const int total = (ui.n - ui.first + kChunkRows - 1) / kChunkRows;
        const int per_seg = ui.seg_rows / kChunkRows;
        int landed = 0;
        bool done = true;
        if (lane < ui.seg) {
            const unsigned long long v = ld_acquire_u64(ui.prog + lane);
            landed = (v >> 32) == (unsigned long long)epoch ? (int)(uint32_t)v : 0;
            done = landed >= min(per_seg, total - lane * per_seg);
        }
        const uint32_t open = __ballot_sync(0xFFFFFFFFu, !done);
        if (open == 0) {
            safe.below = kNoBound;  // everything in front of the segment has landed
        } else {
            // rows in front of J = first row not known to have landed; sources below keep[J]
            // all belong to rows in front of J
            const int g = __ffs(open) - 1;
            const int rows_in = __shfl_sync(0xFFFFFFFFu, landed, g) * kChunkRows;
            int bound = 0;
            if (lane == 0) bound = ui.keep[ui.first + g * ui.seg_rows + rows_in];
            safe.below = __shfl_sync(0xFFFFFFFFu, bound, 0);
        }
        if (d_end <= safe.below) break;
        if (++polls > limit) return false;
        __nanosleep(200);
    }
    return true;
}

// Lane 0 waits for the loads of chunk c and publishes the segment's progress; for a chunk of a
// later segment the warp makes sure no earlier segment still needs the rows the chunk
// overwrites; lane 0 stores the chunk.  Returns false (to all lanes) if a wait ran out.
__device__ __forceinline__ bool store_chunk(uint64_t* full, const StageInfo* info, const UnitInfo* units,
                                            char* buf, int64_t c, int stages, uint32_t stage_bytes,
                                            int lane, uint32_t epoch, SafeBound& safe) {
    const int stage = (int)(c % stages);
    const StageInfo* si = &info[stage];
    int ok = 1;
    if (lane == 0) {
        ok = mbar_wait_bounded(&full[stage], (uint32_t)((c / stages) & 1), kMbarSpinLimit);
        if (ok && si->publish != 0) {
            const UnitInfo* ui = &units[si->unit % kMaxStages];
            st_relaxed_u64(ui->prog + ui->seg, ((unsigned long long)epoch << 32) | si->publish);
        }
    }
    const int32_t d_end = si->d_end;  // the same word for every lane
    if (d_end != 0) {
        ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
        if (ok) {
            const uint32_t unit = si->unit;
            ok = wait_for_earlier_segments(units[unit % kMaxStages], d_end, unit, epoch, safe, lane, kSpinLimit);
        }
    }
    if (lane == 0 && ok) {
        bulk_store(si->dst, buf + (size_t)stage * stage_bytes, si->bytes);
        bulk_commit();
    }
    return __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
}

// One work unit (a segment of the moved rows of one plane), resolved from its number.
struct Unit {
    const char* src;
    char* dst;
    const int32_t* keep;
    unsigned long long* prog;  // progress words of the plane (chained units)
    int j_begin, j_end;        // destination rows of the segment
    int h, n_seg;              // segment index, segments of the plane
    int f, n, seg_rows;        // first moved row, rows kept, rows per full segment
    bool chained;              // in place and the plane has several segments
    bool valid;                // false: nothing to move for this number
};

__device__ __forceinline__ Unit resolve_unit(const CompactParams& p, int64_t u, int units_base, int seg_chunks) {
    Unit un;
    un.h = (int)(u / units_base);  // segment of the plane's moved rows
    const int r = (int)(u - (int64_t)un.h * units_base);
    const int tensor = (int)(r / p.planes_per_tensor);
    const int64_t plane = r - (int64_t)tensor * p.planes_per_tensor;
    const int s = (int)(plane / p.planes_per_stream);
    un.n = min(max(p.n_keep[s], 0), p.keep_stride);
    un.f = p.first_moved[s];
    if (!p.in_place && un.f >= 0) un.f = 0;
    const int total_chunks = un.f >= 0 && un.f < un.n ? (un.n - un.f + kChunkRows - 1) / kChunkRows : 0;
    const int per_seg = seg_chunks;
    un.n_seg = (total_chunks + per_seg - 1) / per_seg;  // non-empty segments
    // invalid: keep list rejected, nothing moves, or a segment behind the stream's last one
    un.valid = un.h < un.n_seg;
    const int c_begin = un.h * per_seg, c_end = min(total_chunks, c_begin + per_seg);
    un.j_begin = un.f + c_begin * kChunkRows;
    un.j_end = min(un.n, un.f + c_end * kChunkRows);
    un.seg_rows = per_seg * kChunkRows;
    un.src = (tensor ? p.src[1] : p.src[0]) + (size_t)plane * p.capacity * p.row_bytes;
    un.dst = (tensor ? p.dst[1] : p.dst[0]) + (size_t)plane * p.capacity * p.row_bytes;
    un.keep = p.keep_idx + (size_t)s * p.keep_stride;
    un.chained = p.in_place && un.n_seg > 1;
    un.prog = p.plane_progress + (un.chained ? (size_t)r * kMaxSplit : 0);
    return un;
}

// One warp waits (bounded) until the ready words of all n_streams streams are up.
__device__ __forceinline__ bool wait_until_ready(const int32_t* ready, int n_streams, int lane) {
    int ok = 1;
    for (int s = lane; s < n_streams && ok; s += 32) {
        uint32_t polls = 0;
        while (ld_acquire_u32(&ready[s]) != 1u) {
            if (++polls > kSpinLimit) {
                ok = 0;
                break;
            }
            if (polls > 64) __nanosleep(100);  // the word usually flips within a few microseconds
        }
    }
    ok = __all_sync(0xFFFFFFFFu, ok);
    __syncwarp();
    return ok != 0;
}

__host__ __device__ inline size_t header_bytes(int n_workers) {
    const size_t h = (size_t)n_workers * kMaxStages * (8 + sizeof(StageInfo) + sizeof(UnitInfo));
    return (h + 127) & ~(size_t)127;
}

__global__ void __launch_bounds__(kMaxWorkers * 32, 1)
compact_kernel(const CompactParams p, const int stages, const int units_base, const int split,
               const int seg_chunks) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int n_workers = blockDim.x >> 5;
    const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t stage_bytes = (uint32_t)kChunkRows * (uint32_t)p.row_bytes;

    // shared memory: [workers][kMaxStages] mbarriers, stage records and unit records (chunks
    // in flight belong to at most `stages` units), then the rings
    uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw) + wid * kMaxStages;
    StageInfo* info =
        reinterpret_cast<StageInfo*>(smem_raw + (size_t)n_workers * kMaxStages * 8) + wid * kMaxStages;
    UnitInfo* units = reinterpret_cast<UnitInfo*>(smem_raw + (size_t)n_workers * kMaxStages *
                                                                 (8 + sizeof(StageInfo))) +
                      wid * kMaxStages;
    size_t header = header_bytes(n_workers);
    char* buf = reinterpret_cast<char*>(smem_raw) + header + (size_t)wid * stages * stage_bytes;

    if (lane == 0) {
        for (int i = 0; i < stages; ++i) mbar_init(&full[i], 1);
        mbar_init_fence();
    }
    __syncwarp();

    // The kernel that precedes this one on the stream (selection, or the check of a caller's
    // keep lists) sets the epoch and the ticket counter before this grid can start, and raises
    // ready[s] as soon as stream s's keep list and counts are out, possibly long before it ends.
    // Under a programmatic dependent launch this grid polls those words instead of waiting for
    // the whole preceding grid, so the gather starts while that kernel finishes its other work.
    // Every stream's word is awaited before anything else that kernel wrote is read (lane i
    // takes streams i, i + 32, ...), so those reads may go through L1.
    const uint32_t epoch = (uint32_t)*p.epoch;
    const int lead = stages - 1 - kStoreSlack;  // chunks whose loads run ahead of the stores
    const int64_t n_units = (int64_t)units_base * split;
    int64_t it = 0;      // chunks whose loads were issued
    int64_t stored = 0;  // chunks whose store was issued
    uint32_t unit_no = 0;
    SafeBound safe;

    // The first numbers are drawn once per CTA for all its workers (a quarter of the counter
    // traffic while the whole grid starts at once), later ones by each worker for itself.
    __shared__ unsigned long long first_ticket;
    if (threadIdx.x == 0) first_ticket = atomicAdd(p.ticket, (unsigned long long)n_workers);
    bool alive = wait_until_ready(p.ready, (int)(p.planes_per_tensor / p.planes_per_stream), lane);
    __syncthreads();
    unsigned long long drawn = first_ticket + wid;  // lane 0's copy counts

    // the unit behind the number lane 0 holds; numbers whose unit is empty are skipped
    auto next_unit = [&]() -> Unit {
        Unit un;
        un.valid = false;
        while (alive) {
            const int64_t u = (int64_t)__shfl_sync(0xFFFFFFFFu, drawn, 0);
            if (u >= n_units) break;
            un = resolve_unit(p, u, units_base, seg_chunks);
            if (un.valid) break;
            if (lane == 0) drawn = atomicAdd(p.ticket, 1ull);
        }
        return un;
    };
    // source rows of a unit's first kIdxAhead chunks, one per lane and chunk
    auto first_indices = [&](const Unit& un, int (&k)[kIdxAhead]) {
#pragma unroll
        for (int q = 0; q < kIdxAhead; ++q) {
            const int j = un.j_begin + q * kChunkRows + lane;
            k[q] = (un.valid && j < un.j_end) ? un.keep[j] : -2;
        }
    };

    // Source indices are always fetched a whole group of chunks ahead, across unit boundaries
    // too: two groups before a unit ends the next number is drawn, one group before the end
    // that unit is resolved and its first indices are requested, so that neither the counter
    // nor the index loads sit on the critical path when the worker moves on.
    Unit cur = next_unit();
    int kq[kIdxAhead];
    first_indices(cur, kq);
    while (alive && cur.valid) {
        ++unit_no;  // counts the units that put chunks into the ring
        if (cur.chained && lane == 0) {
            UnitInfo ui;
            ui.keep = cur.keep;
            ui.prog = cur.prog;
            ui.seg = cur.h;
            ui.first = cur.f;
            ui.seg_rows = cur.seg_rows;
            ui.n = cur.n;
            units[unit_no % kMaxStages] = ui;
        }
        const int j_begin = cur.j_begin, j_end = cur.j_end;
        bool drew = false, resolved = false;
        Unit nxt;
        nxt.valid = false;
        int kq_next[kIdxAhead];
        for (int jg = j_begin; jg < j_end && alive; jg += kIdxAhead * kChunkRows) {
            if (!drew && jg + 2 * kIdxAhead * kChunkRows >= j_end) {
                if (lane == 0) drawn = atomicAdd(p.ticket, 1ull);
                drew = true;
            }
            if (!resolved && jg + kIdxAhead * kChunkRows >= j_end) {
                nxt = next_unit();
                first_indices(nxt, kq_next);
                resolved = true;
            }
            int kn[kIdxAhead];
#pragma unroll
            for (int q = 0; q < kIdxAhead; ++q) {
                const int j = jg + (kIdxAhead + q) * kChunkRows + lane;
                kn[q] = j < j_end ? cur.keep[j] : -2;
            }
#pragma unroll
            for (int q = 0; q < kIdxAhead; ++q) {
                const int j0 = jg + q * kChunkRows;
                if (j0 >= j_end || !alive) break;
                const int nrows = min(kChunkRows, j_end - j0);
                const int stage = (int)(it % stages);
                const int kj = kq[q];
                if (lane == 0) {
                    if (it >= stages) bulk_wait_read<kStoreSlack>();  // the stage's last store has left
                    StageInfo si;
                    si.dst = cur.dst + (size_t)j0 * p.row_bytes;
                    si.bytes = (uint32_t)nrows * p.row_bytes;
                    si.d_end = (cur.chained && cur.h > 0) ? j0 + nrows : 0;
                    si.unit = unit_no;
                    const int done = (j0 - j_begin) / kChunkRows + 1;  // chunks of the segment so far
                    si.publish = (cur.chained && cur.h + 1 < cur.n_seg &&
                                  (done % kPublishEvery == 0 || j0 + kChunkRows >= j_end))
                                     ? (uint32_t)done
                                     : 0u;
                    info[stage] = si;
                    mbar_expect_tx(&full[stage], si.bytes);
                }
                __syncwarp();
                // one bulk load per run of consecutive source rows
                const int prev = __shfl_up_sync(0xFFFFFFFFu, kj, 1);
                const bool head = lane < nrows && (lane == 0 || kj != prev + 1);
                const uint32_t heads = __ballot_sync(0xFFFFFFFFu, head);
                if (head) {
                    const uint32_t later = lane == 31 ? 0u : (heads & ~((2u << lane) - 1u));
                    const int next = later ? __ffs(later) - 1 : nrows;
                    bulk_load(buf + (size_t)stage * stage_bytes + (size_t)lane * p.row_bytes,
                              cur.src + (size_t)kj * p.row_bytes, (uint32_t)(next - lane) * p.row_bytes,
                              &full[stage]);
                }
                ++it;
                if (it - stored > lead) {
                    alive = store_chunk(full, info, units, buf, stored, stages, stage_bytes, lane, epoch, safe);
                    ++stored;
                }
            }
#pragma unroll
            for (int q = 0; q < kIdxAhead; ++q) kq[q] = kn[q];
        }
        cur = nxt;
#pragma unroll
        for (int q = 0; q < kIdxAhead; ++q) kq[q] = kq_next[q];
    }
    while (alive && stored < it) {
        alive = store_chunk(full, info, units, buf, stored, stages, stage_bytes, lane, epoch, safe);
        ++stored;
    }
    if (lane == 0) {
        if (!alive) {
            // a wait ran out: nothing more is stored, but the bulk loads already issued still
            // write into this CTA's shared memory - let them land (bounded) before leaving
            atomicOr(p.status, SIRLLM_STATUS_TIMEOUT);
            for (int64_t c = max(stored - 1, (int64_t)0); c < it; ++c)
                (void)mbar_wait_bounded(&full[c % stages], (uint32_t)((c / stages) & 1), kMbarSpinLimit);
        }
        bulk_wait_all();
        // this grid must not be complete before the one it depends on is (what follows on the
        // stream may rely on both); in practice that kernel ended long ago
        grid_dependency_wait();
    }
}

// Small jobs (a few MB in all: short caches on few planes).  The ring above needs a long run
// of chunks per worker to reach its speed and fills an SM's shared memory per CTA; here one CTA
// takes one column slice of one plane and moves it in two phases - every moved row piece is
// loaded into shared memory with 128-bit loads, the block synchronises, every piece is stored -
// so no store can overtake a load, in place or not, and slices (whole 32-byte sectors of a
// row) never touch each other's bytes.  Chosen by the host when all of a slice fits in shared
// memory and the job is too small to fill the persistent grid.
constexpr int kSmallThreads = 256;

__global__ void __launch_bounds__(kSmallThreads)
compact_small_kernel(const CompactParams p, const int col_splits) {
    extern __shared__ uint4 staged[];
    __shared__ int sh_ok;
    const int r = (int)(blockIdx.x / col_splits), c = (int)(blockIdx.x - (unsigned)r * col_splits);
    const int tensor = (int)(r / p.planes_per_tensor);
    const int64_t plane = r - (int64_t)tensor * p.planes_per_tensor;
    const int s = (int)(plane / p.planes_per_stream);
    if (threadIdx.x < 32) {  // the keep lists are out (see compact_kernel)
        const bool ok = wait_until_ready(p.ready, (int)(p.planes_per_tensor / p.planes_per_stream), threadIdx.x);
        if (threadIdx.x == 0) {
            if (!ok) atomicOr(p.status, SIRLLM_STATUS_TIMEOUT);
            sh_ok = ok;
        }
    }
    __syncthreads();
    if (sh_ok) {
        const int n = min(max(p.n_keep[s], 0), p.keep_stride);
        int f = p.first_moved[s];
        if (!p.in_place && f >= 0) f = 0;
        if (f >= 0 && f < n) {
            const int row_vecs = p.row_bytes / 16, slice_vecs = row_vecs / col_splits;
            const uint4* src = reinterpret_cast<const uint4*>(
                (tensor ? p.src[1] : p.src[0]) + (size_t)plane * p.capacity * p.row_bytes) + c * slice_vecs;
            uint4* dst = reinterpret_cast<uint4*>(
                (tensor ? p.dst[1] : p.dst[0]) + (size_t)plane * p.capacity * p.row_bytes) + c * slice_vecs;
            const int32_t* keep = p.keep_idx + (size_t)s * p.keep_stride;
            const int total = (n - f) * slice_vecs;
            constexpr int kBatch = 4;  // independent loads in flight per thread
            for (int base = 0; base < total; base += kBatch * kSmallThreads) {
                int kj[kBatch];
#pragma unroll
                for (int q = 0; q < kBatch; ++q) {
                    const int i = base + q * kSmallThreads + threadIdx.x;
                    kj[q] = i < total ? keep[f + i / slice_vecs] : 0;
                }
                uint4 x[kBatch];
#pragma unroll
                for (int q = 0; q < kBatch; ++q) {
                    const int i = base + q * kSmallThreads + threadIdx.x;
                    if (i < total) x[q] = src[(size_t)kj[q] * row_vecs + i % slice_vecs];
                }
#pragma unroll
                for (int q = 0; q < kBatch; ++q) {
                    const int i = base + q * kSmallThreads + threadIdx.x;
                    if (i < total) staged[i] = x[q];
                }
            }
            __syncthreads();  // every source row of the slice has been read
            for (int i = threadIdx.x; i < total; i += kSmallThreads)
                dst[(size_t)(f + i / slice_vecs) * row_vecs + i % slice_vecs] = staged[i];
        }
    }
    // a kernel launched programmatically behind this grid (the next round's scorer) may become
    // resident from here on; it waits for the whole grid itself before it reads anything
    grid_launch_dependents();
    // not complete before the grid this one depends on is (see compact_kernel)
    if (threadIdx.x == 0) grid_dependency_wait();
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
        // the same hand-off as the selection kernel's: ready word down, epoch and ticket counter
        // set for the gather, all of it visible before the gather's grid may start
        st_relaxed_u32(&p.ready[s], 0u);
        if (s == 0) {
            *p.epoch += 1;
            *p.ticket = 0ull;
        }
        __threadfence();
    }
    __syncthreads();
    grid_launch_dependents();
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
        __threadfence();
        st_relaxed_u32(&p.ready[s], 1u);  // the gather polls this word
    }
}

// Runs the gather's wait for earlier segments against a progress word that nothing sets (a
// segment of an epoch no compaction reaches), so that it gives up after `limit` polls and
// reports the expiry through the status word: lets a caller check the time-out path on a
// healthy GPU.
__global__ void bounded_wait_selftest_kernel(unsigned long long* prog, const int32_t* keep,
                                             uint32_t limit, int32_t* status) {
    UnitInfo ui;
    ui.keep = keep;  // keep[0] is read: any valid word (rows below it count as safe)
    ui.prog = prog;
    ui.seg = 1;
    ui.first = 0;
    ui.seg_rows = kChunkRows;
    ui.n = 2 * kChunkRows;
    SafeBound safe;
    // a row beyond any slot number, in an epoch no compaction reaches
    const bool ok = wait_for_earlier_segments(ui, kNoBound - 1, 1u, 0xFFFFFFFFu, safe, threadIdx.x & 31, limit);
    if (!ok && threadIdx.x == 0) atomicOr(status, SIRLLM_STATUS_TIMEOUT);
}

}  // namespace

cudaError_t launch_bounded_wait_selftest(unsigned long long* prog, const int32_t* keep, uint32_t limit,
                                         int32_t* status, cudaStream_t st) {
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(prog, keep, limit, status);
    return cudaGetLastError();
}

cudaError_t launch_compact_plan(const CompactParams& p, int n_streams, int32_t* first_moved,
                                cudaStream_t st) {
    TraceRange trace("sirllm:compact_plan");
    compact_plan_kernel<<<n_streams, 256, 0, st>>>(p, first_moved);
    return cudaGetLastError();
}

bool compact_is_small_job(int64_t planes, int keep_stride, int row_bytes) {
    return planes * keep_stride * row_bytes <= kSmallJobBytes;
}

cudaError_t launch_compact(const CompactParams& p, cudaStream_t st, bool overlap) {
    TraceRange trace("sirllm:compact_kv");
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
    if (units64 > 0x3FFFFFFF) return cudaErrorInvalidValue;
    const int units_base = (int)units64;

    DeviceProps dp;
    cudaError_t e = device_props(&dp);
    if (e != cudaSuccess) return e;
    const int n_sm = dp.n_sm, smem_max = dp.smem_optin;
    static unsigned char allowed_ring[kMaxDevices], allowed_small[kMaxDevices];

    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;

    // a job too small to fill the persistent grid goes to the two-phase kernel: one CTA per
    // plane and column slice (slices of at least 32 bytes, as many as it takes to occupy the
    // SMs), provided a slice of the longest keep list fits in shared memory
    const int row_vecs = p.row_bytes / 16;
    if (compact_is_small_job(units_base, p.keep_stride, p.row_bytes)) {
        int col_splits = 1;
        while (col_splits * 2 <= row_vecs / 2 && row_vecs % (col_splits * 2) == 0 &&
               (int64_t)units_base * col_splits < 2 * n_sm)
            col_splits *= 2;
        const size_t small_smem = (size_t)p.keep_stride * (p.row_bytes / col_splits);
        if (small_smem <= (size_t)smem_max - 1024) {
            e = allow_max_dynamic_smem((const void*)compact_small_kernel, dp, allowed_small);
            if (e != cudaSuccess) return e;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)(units_base * col_splits));
            cfg.blockDim = dim3(kSmallThreads);
            cfg.dynamicSmemBytes = small_smem;
            cfg.stream = st;
            cfg.attrs = attr;
            cfg.numAttrs = overlap ? 1 : 0;
            return cudaLaunchKernelEx(&cfg, compact_small_kernel, q, col_splits);
        }
    }

    // ring geometry: kMaxWorkers workers per CTA with 6 to 8 stages each; fewer workers, then
    // fewer stages (at least 4), when the rows are too wide for that
    const size_t stage_bytes = (size_t)kChunkRows * p.row_bytes;
    // what is left for the rings beside the records in front of them and the kernel's few
    // bytes of static shared memory
    const size_t budget = (size_t)smem_max - header_bytes(kMaxWorkers) - 256;
    int workers = kMaxWorkers, stages = 6;
    while (workers > 1 && (size_t)workers * stages * stage_bytes > budget) --workers;
    while (stages > 4 && (size_t)workers * stages * stage_bytes > budget) --stages;
    if ((size_t)workers * stages * stage_bytes > budget) return cudaErrorInvalidValue;
    while (stages < 8 && (size_t)workers * (stages + 1) * stage_bytes <= budget) ++stages;
    const size_t smem = header_bytes(workers) + (size_t)workers * stages * stage_bytes;
    e = allow_max_dynamic_smem((const void*)compact_kernel, dp, allowed_ring);
    if (e != cudaSuccess) return e;

    // a persistent grid: as many CTAs as the device keeps resident at once (the ring fills an
    // SM's shared memory, so one per SM), fewer when there is less work.  The occupancy of a
    // geometry is asked of the runtime once per device and remembered.
    static std::atomic<long long> occ_cache[kMaxDevices];  // (smem << 20 | workers << 8 | per_sm) + 1
    const long long occ_key = ((long long)smem << 20) | ((long long)workers << 8);
    int per_sm = 0;
    const bool slot = dp.device >= 0 && dp.device < kMaxDevices;
    const long long seen = slot ? occ_cache[dp.device].load(std::memory_order_acquire) - 1 : -1;
    if (seen >= 0 && (seen & ~0xFFll) == occ_key) {
        per_sm = (int)(seen & 0xFF);
    } else {
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, compact_kernel, workers * 32, smem);
        if (e != cudaSuccess) return e;
        if (slot) occ_cache[dp.device].store((occ_key | (per_sm & 0xFF)) + 1, std::memory_order_release);
    }
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    const int64_t resident = (int64_t)n_sm * per_sm;
    // Cut planes into segments so that every worker draws a dozen or two units: the ticket
    // hand-out then evens out SMs of different speed down to a small tail, while a unit stays
    // long enough to amortise its set-up.  Segments are a fixed number of chunks long
    // (`seg_chunks`), chosen ODD: planes are a power of two apart, so segments of 2^k chunks
    // would make all workers walk addresses that differ by large powers of two at the same
    // time, which measured 2-3 % slower than odd lengths around the same size.  About 16 units
    // per worker measured best over the shapes tried: with 2048 planes of 64 chunks (planes 1 MB
    // apart) segments of 15 to 21 chunks are 4-5 % faster than segments of 7; elsewhere 10 to 30
    // units per worker are within a percent, below 7 the tail shows.  The last, shorter segment
    // of every plane is handed out last and keeps that tail fine.
    const int64_t slots = resident * workers;
    const int64_t chunks_max = (p.keep_stride + kChunkRows - 1) / kChunkRows;
    int64_t seg_chunks = chunks_max;  // one segment per plane
    if (units_base <= kChainPlanesMax) {
        // chunks of all planes shared out over kUnitsPerWorker units per worker
        int64_t want = (chunks_max * units_base + kUnitsPerWorker * slots / 2) / (kUnitsPerWorker * slots);
        if (want < kMinSegChunks) want = kMinSegChunks;
        if (want % 2 == 0) ++want;
        const int64_t least = (chunks_max + kMaxSplit - 1) / kMaxSplit;  // at most kMaxSplit segments
        if (want < least) want = least;
        if (want < chunks_max) seg_chunks = want;
    }
    const int split = (int)((chunks_max + seg_chunks - 1) / seg_chunks);
    const int64_t n_units = (int64_t)units_base * split;
    const int64_t want = (n_units + workers - 1) / workers;
    const int grid = (int)(want < resident ? want : resident);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)workers * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, compact_kernel, q, stages, units_base, split, (int)seg_chunks);
}

}  // namespace sirllm
