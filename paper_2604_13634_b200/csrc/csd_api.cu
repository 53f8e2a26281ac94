// C ABI of the CSD verification library (see include/csd.h for the contract).
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <algorithm>
#include <cstring>
#include <mutex>
#include <vector>
#include <new>

#include "../../include/csd.h"
#include "csd_common.cuh"
#include "csd_ocm.cuh"
#include "csd_step.cuh"
#include "csd_sampled.cuh"
#include "csd_lmhead.cuh"

using namespace csd;

struct csd_ocm {
    int device;
    uint64_t n_slots;
    uint32_t lambda;
    OcmSlot *slots;
    OcmStatsDev *stats;
    int shared;                     // csd_ocm_set_shared
    unsigned long long *age_keys;   // side arrays of csd_ocm_age: n_slots / 2 entries each
    unsigned int *age_counts;
};

namespace {

constexpr int kDefaultSms = 148;   // B200; used only when no device can be queried
constexpr int kMaxLmheadDevices = 64;

int g_chunk_bytes_override = 0;
int g_ctas_per_sm_override = 0;
int g_block_threads_override = 0;
int g_overlap_steps = 0;

// ---- which launch preceded which ----------------------------------------------------------
// A step launched with overlap may poll the completion count that the previous step leaves in
// the workspace instead of waiting for that whole grid to retire -- but only if that previous
// step launch on the stream really was issued with the same workspace, memory, outputs and
// shape, and nothing of this library touched them since.  The host keeps the last step launch
// per stream for that; any other call that launches work or changes the layout starts a new
// generation, which voids every record.
struct ChainRecord {
    void *stream;
    const void *ws, *ocm, *out;
    int B, K, V, dtype;
    unsigned long long generation;
};
constexpr int kChainRecords = 16;
std::mutex g_chain_mutex;
ChainRecord g_chain[kChainRecords];
int g_chain_used = 0, g_chain_next = 0;
unsigned long long g_chain_generation = 1;

void chain_break()
{
    std::lock_guard<std::mutex> lock(g_chain_mutex);
    ++g_chain_generation;
}

// Records this launch as the stream's latest; true if the stream's previous record matches it.
bool chain_follows(void *stream, const void *ws, const void *ocm, const void *out, int B, int K, int V, int dtype)
{
    std::lock_guard<std::mutex> lock(g_chain_mutex);
    const ChainRecord now = {stream, ws, ocm, out, B, K, V, dtype, g_chain_generation};
    for (int i = 0; i < g_chain_used; ++i) {
        ChainRecord &r = g_chain[i];
        if (r.stream != stream) continue;
        const bool same = r.ws == ws && r.ocm == ocm && r.out == out && r.B == B && r.K == K && r.V == V &&
                          r.dtype == dtype && r.generation == g_chain_generation;
        r = now;
        return same;
    }
    if (g_chain_used < kChainRecords) {
        g_chain[g_chain_used++] = now;
    } else {
        g_chain[g_chain_next] = now;
        g_chain_next = (g_chain_next + 1) % kChainRecords;
    }
    return false;
}

// ---- which layout a workspace currently holds -----------------------------------------------
// The scratch layout inside a workspace depends on the launch shape (grid, partial slots per
// row), and so on csd_set_overlap / csd_set_tuning as well as on (B, K, V, dtype).  A workspace
// whose counters were left by steps of another layout must be cleared before a step of this
// layout touches it: its tickets would otherwise start from stale words and no row would ever
// be finalised.  The host remembers, per workspace address, the layout of the last step issued
// on it; a step that finds another layout (or no record) enqueues a clear first.
struct WorkspaceRecord {
    const void *ws;
    size_t bytes;               // bytes the recorded layout covers
    unsigned long long sig[3];  // layout signature
    unsigned long long age;
};
constexpr int kWorkspaceRecords = 64;
WorkspaceRecord g_ws_records[kWorkspaceRecords];
int g_ws_used = 0;
unsigned long long g_ws_clock = 0;

// True if `ws` is known to hold exactly this layout; records it otherwise (caller clears).
bool workspace_holds(const void *ws, size_t bytes, const unsigned long long (&sig)[3])
{
    std::lock_guard<std::mutex> lock(g_chain_mutex);
    ++g_ws_clock;
    int victim = 0;
    for (int i = 0; i < g_ws_used; ++i) {
        WorkspaceRecord &r = g_ws_records[i];
        if (r.ws == ws) {
            const bool same = r.bytes == bytes && r.sig[0] == sig[0] && r.sig[1] == sig[1] && r.sig[2] == sig[2];
            r.bytes = bytes;
            r.sig[0] = sig[0]; r.sig[1] = sig[1]; r.sig[2] = sig[2];
            r.age = g_ws_clock;
            return same;
        }
        if (r.age < g_ws_records[victim].age) victim = i;
    }
    if (g_ws_used < kWorkspaceRecords) victim = g_ws_used++;
    WorkspaceRecord &r = g_ws_records[victim];
    r.ws = ws;
    r.bytes = bytes;
    r.sig[0] = sig[0]; r.sig[1] = sig[1]; r.sig[2] = sig[2];
    r.age = g_ws_clock;
    return false;
}

// Forget every record that overlaps [ws, ws + bytes): the range was cleared or is about to be reused.
void workspace_forget(const void *ws, size_t bytes)
{
    std::lock_guard<std::mutex> lock(g_chain_mutex);
    const char *lo = static_cast<const char *>(ws), *hi = lo + bytes;
    for (int i = 0; i < g_ws_used;) {
        const char *a = static_cast<const char *>(g_ws_records[i].ws);
        if (a < hi && a + g_ws_records[i].bytes > lo)
            g_ws_records[i] = g_ws_records[--g_ws_used];
        else
            ++i;
    }
}

int sm_count()
{
    static int cached = 0;
    if (cached > 0) return cached;
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) {
        cached = n;
        return n;
    }
    (void)cudaGetLastError();
    return kDefaultSms;
}

struct Shape {
    int grid;              // blocks = spans of the unit space
    int block;             // threads per block
    int unit_elems;        // elements per 512-byte unit
    int units_per_row;
    int slots_per_row;     // partial slots reserved per logit row
    int chunk_units;       // units per chunk of the in-block hand-out
    long long total_units;
};

inline int elt_bytes(csd_dtype_t dt) { return dt == CSD_F32 ? 4 : 2; }

constexpr int kUnitBytes = 512;   // one 16-byte vector per lane

bool shape_ok(int B, int K, int V, csd_dtype_t dt)
{
    if (!(B > 0 && K > 0 && V > 0 && K <= CSD_MAX_K && (dt == CSD_F32 || dt == CSD_BF16))) return false;
    // row and position indices are 32-bit
    return static_cast<long long>(B) * (K + 1) < (1ll << 31) && static_cast<long long>(B) * K < (1ll << 31);
}

// The unit space (R rows x U units of 512 bytes) is split evenly over the blocks of a
// persistent grid, but no more than 64 blocks per row (few partials per row keep the last
// fold short), at least ~8 KiB each, never more than units.  Blocks per SM: a launch that
// runs alone needs the whole machine (4 blocks per SM, all that fit); with step overlap
// several launches are resident at once and share it, and one block per SM and launch
// lets the next launches start while this one is still streaming (measured: 1 is best on
// every reference workload, 4 costs 15 to 50 % there).
Shape pick_shape(int B, int K, int V, csd_dtype_t dt, bool overlap)
{
    const int eb = elt_bytes(dt);
    const int ctas_per_sm = g_ctas_per_sm_override > 0 ? g_ctas_per_sm_override : (overlap ? 1 : 4);
    const long long rows = static_cast<long long>(B) * (K + 1);
    Shape s;
    s.block = g_block_threads_override > 0 ? g_block_threads_override : kThreads;
    s.unit_elems = kUnitBytes / eb;
    s.units_per_row = (V + s.unit_elems - 1) / s.unit_elems;
    s.total_units = rows * s.units_per_row;
    long long blocks = static_cast<long long>(sm_count()) * ctas_per_sm;
    if (blocks > rows * 64) blocks = rows * 64;
    // at least 8 KiB per block; for a launch that runs alone 32 KiB (one full iteration for each of eight
    // warps): below that more blocks only mean more partial results to exchange and fold at the end
    const long long min_units = overlap ? 16 : 64;
    if (blocks > (s.total_units + min_units - 1) / min_units) blocks = (s.total_units + min_units - 1) / min_units;
    if (blocks < 1) blocks = 1;
    s.grid = static_cast<int>(blocks);
    // span boundaries lie at floor(c*T/G): at most ceil((U-1)*G/T) of them fall inside a row
    long long slots = ((s.units_per_row - 1) * blocks + s.total_units - 1) / s.total_units + 1;
    if (slots > s.units_per_row) slots = s.units_per_row;
    s.slots_per_row = static_cast<int>(slots < 1 ? 1 : slots);
    // chunks: about one per warp of the block for small spans (least per-chunk overhead), 4 to
    // 32 KiB in whole warp iterations (4 KiB), so that larger spans are still handed out in many
    // pieces; grown where needed so that a block's span fits its chunk table
    const long long span_max = (s.total_units + blocks - 1) / blocks;
    const int warps = s.block / 32;
    long long chunk_units = ((span_max + warps - 1) / warps + 7) / 8 * 8;
    if (chunk_units < 8) chunk_units = 8;
    if (chunk_units > 64) chunk_units = 64;
    if (g_chunk_bytes_override > 0) chunk_units = g_chunk_bytes_override / kUnitBytes;
    const long long need = (span_max + (kMaxChunks - kMaxSegs - 2) - 1) / (kMaxChunks - kMaxSegs - 2);
    if (chunk_units < need) chunk_units = (need + 7) / 8 * 8;
    s.chunk_units = static_cast<int>(chunk_units);
    return s;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct WorkspaceLayout {
    size_t seq_off, copy_bytes, partials_off, hint_off, b_ticket_off, g_ticket_off, total;   // *_off within a copy
};

// header {launch sequence, blocks counted in, launches completed} followed by kScratchRing copies of the scratch,
// each {partials | slot hints | per-batch-row tickets | global ticket}
WorkspaceLayout ws_layout(int B, int K, const Shape &s)
{
    WorkspaceLayout w;
    w.seq_off = 0;
    w.partials_off = 0;
    w.hint_off = align_up(static_cast<size_t>(B) * (K + 1) * s.slots_per_row * sizeof(Partial), 256);
    w.b_ticket_off = align_up(w.hint_off + static_cast<size_t>(B) * K * sizeof(int), 256);
    w.g_ticket_off = align_up(w.b_ticket_off + static_cast<size_t>(B) * sizeof(unsigned int), 16);
    w.copy_bytes = align_up(w.g_ticket_off + 16, 256);
    w.total = 256 + kScratchRing * w.copy_bytes;
    return w;
}

OcmView view_of(const csd_ocm *o)
{
    OcmView v;
    v.slots = o->slots;
    v.mask = o->n_slots - 1;
    v.key_limit = o->n_slots / 2;
    v.lambda = o->lambda;
    v.stats = o->stats;
    v.shared = o->shared;
    return v;
}

// A launch that covers positions pos0 .. pos0 + K - 1 of a step with K_total positions, on all batch rows or on
// the rows listed in device memory (the two phases of csd_step_early_exit).
struct PhaseSpec {
    int K_total, pos0;
    const int *row_map, *n_rows;
    int *alive_out, *n_alive_out;
    int count_positions, count_step;
};

constexpr int kListSlotsPerRow = 66;   // a launch over a row list may put up to 64 blocks (+ 2 boundary blocks) on a logit row

csd_status_t run_step(const void *logits, csd_dtype_t dtype, int B, int K, int V, int64_t stride_b, int64_t stride_k,
                      const int32_t *draft, const csd_ocm *ocm, float tau, int32_t *accept_len, int32_t *next_token,
                      uint8_t *rescued_mask, int32_t *rej_draft, int32_t *rej_target, const csd_diag_t *diag,
                      void *workspace, size_t workspace_bytes, void *stream, bool do_update, bool may_chain = true,
                      bool may_overlap = true, bool track_layout = true, const PhaseSpec *phase = nullptr)
{
    if (!logits || !draft || !ocm || !accept_len || !next_token || !rescued_mask || !rej_draft || !rej_target || !workspace)
        return CSD_ERR_INVALID_ARG;
    if (B <= 0 || K <= 0 || V <= 0) return CSD_ERR_INVALID_ARG;
    if (dtype != CSD_F32 && dtype != CSD_BF16) return CSD_ERR_INVALID_ARG;
    if (K > CSD_MAX_K) return CSD_ERR_UNSUPPORTED;
    if (!shape_ok(B, K, V, dtype)) return CSD_ERR_UNSUPPORTED;
    if (!(tau >= 0.0f) || std::isinf(tau)) return CSD_ERR_INVALID_ARG;   // also refuses NaN
    if (stride_k < V || stride_b < stride_k * ((phase ? phase->K_total : K) + 1)) return CSD_ERR_INVALID_ARG;

    Shape s = pick_shape(B, K, V, dtype, g_overlap_steps != 0 && may_overlap);
    if (phase && phase->n_rows) s.slots_per_row = s.units_per_row < kListSlotsPerRow ? s.units_per_row : kListSlotsPerRow;
    const WorkspaceLayout w = ws_layout(B, K, s);
    if (workspace_bytes < w.total || (reinterpret_cast<uintptr_t>(workspace) & 15u)) return CSD_ERR_WORKSPACE;

    StepParams p;
    std::memset(&p, 0, sizeof p);
    p.logits = logits;
    p.B = B; p.K = K; p.V = V;
    p.stride_b = stride_b; p.stride_k = stride_k;
    p.draft = draft;
    p.ocm = view_of(ocm);
    p.log_tau = csd_scg_threshold(tau);
    p.do_update = do_update ? 1 : 0;
    p.accept_len = accept_len; p.next_token = next_token; p.rescued = rescued_mask;
    p.rej_d = rej_draft; p.rej_t = rej_target;
    if (diag) p.diag = *diag;
    char *ws = static_cast<char *>(workspace);
    if (w.copy_bytes > 0xffffffffull) return CSD_ERR_UNSUPPORTED;
    p.scratch = ws + 256;
    p.copy_bytes = static_cast<unsigned int>(w.copy_bytes);
    p.hint_off = static_cast<unsigned int>(w.hint_off);
    p.b_ticket_off = static_cast<unsigned int>(w.b_ticket_off);
    p.g_ticket_off = static_cast<unsigned int>(w.g_ticket_off);
    p.launch_seq = reinterpret_cast<unsigned long long *>(ws + w.seq_off);
    p.completed = reinterpret_cast<unsigned int *>(ws + w.seq_off + 8);
    p.n_spans = s.grid;
    p.unit_elems = s.unit_elems;
    p.units_per_row = s.units_per_row;
    p.slots_per_row = s.slots_per_row;
    p.chunk_units = s.chunk_units;
    p.total_units = s.total_units;
    p.narrow = ((s.total_units + 1) * (static_cast<long long>(s.grid) + 1) < (1ll << 32) && s.total_units * 40 < (1ll << 32)) ? 1 : 0;
    if (phase) {
        p.K_total = phase->K_total;
        p.pos0 = phase->pos0;
        p.row_map = phase->row_map;
        p.n_rows = phase->n_rows;
        p.alive_out = phase->alive_out;
        p.n_alive_out = phase->n_alive_out;
        p.count_positions = phase->count_positions;
        p.count_step = phase->count_step;
        p.min_units = (g_overlap_steps != 0 && may_overlap) ? 16 : 64;
    }
    if (track_layout) {
        const unsigned long long sig[3] = {
            (static_cast<unsigned long long>(static_cast<unsigned int>(B)) << 32) | static_cast<unsigned int>(K),
            (static_cast<unsigned long long>(static_cast<unsigned int>(s.grid)) << 32) | static_cast<unsigned int>(s.slots_per_row),
            (static_cast<unsigned long long>(w.copy_bytes) << 8) | static_cast<unsigned int>(dtype)};
        if (!workspace_holds(workspace, w.total, sig)) {
            // first step of this layout on this workspace: start from cleared counters
            chain_break();
            if (cudaMemsetAsync(workspace, 0, w.total, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
                (void)cudaGetLastError();
                workspace_forget(workspace, w.total);
                return CSD_ERR_CUDA;
            }
        }
    }
    const bool follows = chain_follows(stream, workspace, ocm, accept_len, B, K, V, static_cast<int>(dtype));
    p.chain_by_flag = (may_chain && follows) ? 1 : 0;
    p.stream_ordered = (g_overlap_steps && may_overlap) ? 0 : 1;

    const int eb = elt_bytes(dtype);
    const int per_vec = 16 / eb;
    const bool vec = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && (stride_b * eb) % 16 == 0 &&
                     (stride_k * eb) % 16 == 0 && V % per_vec == 0;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(s.grid);
    cfg.blockDim = dim3(s.block);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    if (g_overlap_steps && may_overlap) {
        // let this launch begin while the previous kernel on the stream drains; the kernel
        // itself waits for that kernel before its first write
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    cudaError_t err;
    if (dtype == CSD_F32) {
        err = vec ? cudaLaunchKernelEx(&cfg, csd_step_kernel<LaneF32Vec>, p)
                  : cudaLaunchKernelEx(&cfg, csd_step_kernel<LaneF32Scalar>, p);
    } else {
        err = vec ? cudaLaunchKernelEx(&cfg, csd_step_kernel<LaneBf16Vec>, p)
                  : cudaLaunchKernelEx(&cfg, csd_step_kernel<LaneBf16Scalar>, p);
    }
    if (err != cudaSuccess) {
        (void)cudaGetLastError();
        chain_break();
        workspace_forget(workspace, w.total);
        return CSD_ERR_CUDA;
    }
    return cudaGetLastError() == cudaSuccess ? CSD_OK : CSD_ERR_CUDA;
}

csd_status_t run_update(csd_ocm *ocm, const int32_t *d, const int32_t *t, const uint32_t *w, int64_t n, void *stream,
                        bool programmatic = false)
{
    if (!ocm || n < 0 || (n > 0 && (!d || !t))) return CSD_ERR_INVALID_ARG;
    if (n == 0) return CSD_OK;
    chain_break();
    long long blocks = (n + 1023) / 1024;
    const long long cap = static_cast<long long>(sm_count()) * 2;
    if (blocks > cap) blocks = cap;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned int>(blocks));
    cfg.blockDim = dim3(1024);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    if (programmatic) {     // behind the kernel that writes d / t: the update kernel waits for it itself
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    const long long n_ll = n;
    if (cudaLaunchKernelEx(&cfg, ocm_update_kernel, view_of(ocm), d, t, w, n_ll) != cudaSuccess) {
        (void)cudaGetLastError();
        return CSD_ERR_CUDA;
    }
    return cudaGetLastError() == cudaSuccess ? CSD_OK : CSD_ERR_CUDA;
}

}  // namespace

// ---- stochastic verification (Algorithm 1 at T > 0) ----------------------------------------
namespace {

constexpr int kSampledChunkMax = 8192;   // most elements of a row reduced by a warp at a time
constexpr int kSampledChunkMin = 2048;   // least (one unrolled iteration of a warp of bf16 vectors)

// Elements per tile: as large as possible while the step still has a few tiles per resident warp.
int sampled_chunk_elems(int B, int K, int V)
{
    const long long rows = static_cast<long long>(B) * (2 * K + 1);
    const long long want = static_cast<long long>(sm_count()) * 32 * 2;
    int chunk = kSampledChunkMax;
    while (chunk > kSampledChunkMin && rows * ((V + chunk - 1) / chunk) < want) chunk /= 2;
    return chunk;
}

struct SampledLayout {
    size_t stat_part, rownorm, alpha, accepted, race_best, row_state, total;
    int nchunks, chunk_elems, race_nchunks;
};

SampledLayout sampled_layout(int B, int K, int V)
{
    SampledLayout w;
    w.chunk_elems = sampled_chunk_elems(B, K, V);
    w.nchunks = (V + w.chunk_elems - 1) / w.chunk_elems;
    w.race_nchunks = (V + kSampledChunkMin - 1) / kSampledChunkMin;
    const size_t rows = static_cast<size_t>(B) * (2 * K + 1);
    const size_t draws = static_cast<size_t>(B) * (K + 1);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t at = off;
        off = align_up(off + bytes, 256);
        return at;
    };
    w.stat_part = take(rows * w.nchunks * sizeof(Partial));
    w.rownorm = take(rows * sizeof(RowNorm));
    w.alpha = take(static_cast<size_t>(B) * K * sizeof(float));
    w.accepted = take(static_cast<size_t>(B) * K);
    w.race_best = take(draws * sizeof(unsigned long long));
    w.row_state = take(static_cast<size_t>(B));
    w.total = off;
    return w;
}

int g_sampled_rounds = 0;             // 0 = automatic, 1 = every draw in one round, 2 = two rounds of draws on demand
// measured: one round takes 26.5 us against 28.9 at 4 MB (single_stream), the same at 107 MB, 28 % longer at 272 MB
constexpr double kSampledSingleRoundBytes = 32e6;

// One round of draws instead of two for steps whose two logit tensors are smaller than this many bytes.
bool sampled_single_round(int B, int K, int V, size_t elt)
{
    if (g_sampled_rounds == 1) return true;
    if (g_sampled_rounds == 2) return false;
    return static_cast<double>(B) * (2 * K + 1) * V * static_cast<double>(elt) < kSampledSingleRoundBytes;
}

template <typename L>
cudaError_t launch_sampled(const SampledParams &p, cudaStream_t st)
{
    const long long rows = static_cast<long long>(p.B) * (2 * p.K + 1);
    const long long draws = static_cast<long long>(p.B) * (p.K + 1);
    const long long cap = static_cast<long long>(sm_count()) * 4;
    auto blocks_for = [&](long long tiles) {
        long long b = (tiles + 7) / 8;            // 8 warps per block
        return static_cast<unsigned int>(b < 1 ? 1 : (b > cap ? cap : b));
    };
    auto launch = [&](auto kernel, unsigned int grid, unsigned int block, bool programmatic, auto... extra) {
        cudaLaunchConfig_t cfg;
        std::memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(block);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        if (programmatic) {
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
        }
        return cudaLaunchKernelEx(&cfg, kernel, p, extra...);
    };
    // The statistics kernel touches only inputs and its own partials before it waits, so it may run
    // beside the previous kernels on the stream when the caller has allowed step overlap; the other
    // three depend on their predecessor alone and wait for it first thing.
    cudaError_t err = launch(sampled_stats_kernel<L>, blocks_for(rows * p.nchunks), 256, g_overlap_steps != 0);
    if (err == cudaSuccess) err = launch(sampled_decide_kernel<L>, static_cast<unsigned int>((draws + 3) / 4), 128, true);
    // two rounds of draws: each row's first failed position (or its bonus row), then what the rows whose
    // first failure was rescued still need; a round's race launch is sized for the draws it can have
    const unsigned int fin_blocks = static_cast<unsigned int>((p.B + 3) / 4);
    if (sampled_single_round(p.B, p.K, p.V, sizeof(typename L::elem))) {
        // a small step: two more launches cost more than the draws that on-demand rounds would save
        if (err == cudaSuccess) err = launch(sampled_race_kernel<L>, blocks_for(draws * p.race_nchunks), 256, true, 0);
        if (err == cudaSuccess) err = launch(sampled_finalize_kernel<L>, fin_blocks, 128, true, 0);
        return err;
    }
    if (err == cudaSuccess) err = launch(sampled_race_kernel<L>, blocks_for(static_cast<long long>(p.B) * p.race_nchunks), 256, true, 1);
    if (err == cudaSuccess) err = launch(sampled_finalize_kernel<L>, fin_blocks, 128, true, 1);
    if (err == cudaSuccess) err = launch(sampled_race_kernel<L>, blocks_for(draws * p.race_nchunks), 256, true, 2);
    if (err == cudaSuccess) err = launch(sampled_finalize_kernel<L>, fin_blocks, 128, true, 2);
    return err;
}

csd_status_t run_sampled(const void *logits, const void *draft_logits, csd_dtype_t dtype, int B, int K, int V,
                         int64_t stride_b, int64_t stride_k, int64_t dstride_b, int64_t dstride_k, const int32_t *draft,
                         const float *r_accept, uint64_t seed, float temperature, csd_ocm *ocm, float tau,
                         int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask, int32_t *rej_draft,
                         int32_t *rej_target, const csd_sampled_diag_t *diag, void *workspace, size_t workspace_bytes,
                         void *stream, bool do_update)
{
    if (!logits || !draft_logits || !draft || !r_accept || !ocm || !accept_len || !next_token || !rescued_mask ||
        !rej_draft || !rej_target || !workspace)
        return CSD_ERR_INVALID_ARG;
    if (B <= 0 || K <= 0 || V <= 0) return CSD_ERR_INVALID_ARG;
    if (dtype != CSD_F32 && dtype != CSD_BF16) return CSD_ERR_INVALID_ARG;
    if (K > CSD_MAX_K) return CSD_ERR_UNSUPPORTED;
    if (!shape_ok(B, K, V, dtype) || static_cast<long long>(B) * (2 * K + 1) >= (1ll << 31)) return CSD_ERR_UNSUPPORTED;
    if (!(tau >= 0.0f) || std::isinf(tau)) return CSD_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || std::isinf(temperature)) return CSD_ERR_INVALID_ARG;
    if (stride_k < V || stride_b < stride_k * (K + 1) || dstride_k < V || dstride_b < dstride_k * K) return CSD_ERR_INVALID_ARG;
    const SampledLayout w = sampled_layout(B, K, V);
    if (workspace_bytes < w.total || (reinterpret_cast<uintptr_t>(workspace) & 15u)) return CSD_ERR_WORKSPACE;
    chain_break();

    SampledParams p;
    std::memset(&p, 0, sizeof p);
    p.z = logits; p.y = draft_logits;
    p.B = B; p.K = K; p.V = V;
    p.z_sb = stride_b; p.z_sk = stride_k; p.y_sb = dstride_b; p.y_sk = dstride_k;
    p.draft = draft; p.r = r_accept;
    p.seed_lo = static_cast<unsigned int>(seed & 0xffffffffull);
    p.seed_hi = static_cast<unsigned int>(seed >> 32);
    p.l2e_T = static_cast<float>(1.4426950408889634 / static_cast<double>(temperature));
    p.ocm = view_of(ocm);
    p.log_tau = csd_scg_threshold(tau);
    p.accept_len = accept_len; p.next_token = next_token; p.rescued = rescued_mask;
    p.rej_d = rej_draft; p.rej_t = rej_target;
    if (diag) p.diag = *diag;
    char *ws = static_cast<char *>(workspace);
    p.stat_part = reinterpret_cast<Partial *>(ws + w.stat_part);
    p.rownorm = reinterpret_cast<RowNorm *>(ws + w.rownorm);
    p.alpha = reinterpret_cast<float *>(ws + w.alpha);
    p.accepted = reinterpret_cast<unsigned char *>(ws + w.accepted);
    p.race_best = reinterpret_cast<unsigned long long *>(ws + w.race_best);
    p.row_state = reinterpret_cast<unsigned char *>(ws + w.row_state);
    p.chunk_elems = w.chunk_elems;
    p.nchunks = w.nchunks;
    p.race_chunk_elems = kSampledChunkMin;
    p.race_nchunks = w.race_nchunks;

    const int eb = elt_bytes(dtype);
    const int per_vec = 16 / eb;
    auto aligned = [&](const void *base, int64_t sb, int64_t sk) {
        return (reinterpret_cast<uintptr_t>(base) % 16 == 0) && (sb * eb) % 16 == 0 && (sk * eb) % 16 == 0;
    };
    const bool vec = aligned(logits, stride_b, stride_k) && aligned(draft_logits, dstride_b, dstride_k) && V % per_vec == 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t err;
    if (dtype == CSD_F32)
        err = vec ? launch_sampled<LaneF32Vec>(p, st) : launch_sampled<LaneF32Scalar>(p, st);
    else
        err = vec ? launch_sampled<LaneBf16Vec>(p, st) : launch_sampled<LaneBf16Scalar>(p, st);
    if (err != cudaSuccess) {
        (void)cudaGetLastError();
        return CSD_ERR_CUDA;
    }
    if (do_update) return run_update(ocm, rej_draft, rej_target, nullptr, static_cast<int64_t>(B) * K, stream, true);
    return CSD_OK;
}

}  // namespace

extern "C" {

csd_status_t csd_ocm_create(csd_ocm_t **out, uint64_t n_slots, uint32_t lambda, int device)
{
    if (!out) return CSD_ERR_INVALID_ARG;
    *out = nullptr;
    if (n_slots < 64 || (n_slots & (n_slots - 1)) != 0 || n_slots > (1ull << 30)) return CSD_ERR_INVALID_ARG;
    if (cudaSetDevice(device) != cudaSuccess) {
        (void)cudaGetLastError();
        return CSD_ERR_CUDA;
    }
    csd_ocm *o = new (std::nothrow) csd_ocm;
    if (!o) return CSD_ERR_OOM;
    o->device = device;
    o->n_slots = n_slots;
    o->lambda = lambda;
    o->shared = 0;
    o->slots = nullptr;
    o->stats = nullptr;
    o->age_keys = nullptr;
    o->age_counts = nullptr;
    if (cudaMalloc(&o->slots, n_slots * sizeof(OcmSlot)) != cudaSuccess ||
        cudaMalloc(&o->stats, sizeof(OcmStatsDev)) != cudaSuccess ||
        cudaMalloc(&o->age_keys, n_slots / 2 * sizeof(unsigned long long)) != cudaSuccess ||
        cudaMalloc(&o->age_counts, n_slots / 2 * sizeof(unsigned int)) != cudaSuccess) {
        (void)cudaGetLastError();
        cudaFree(o->slots);
        cudaFree(o->stats);
        cudaFree(o->age_keys);
        cudaFree(o->age_counts);
        (void)cudaGetLastError();
        delete o;
        return CSD_ERR_OOM;
    }
    csd_status_t rc = csd_ocm_reset(o, nullptr);
    if (rc == CSD_OK && cudaDeviceSynchronize() != cudaSuccess) rc = CSD_ERR_CUDA;
    if (rc != CSD_OK) {
        cudaFree(o->slots);
        cudaFree(o->stats);
        cudaFree(o->age_keys);
        cudaFree(o->age_counts);
        delete o;
        return rc;
    }
    *out = o;
    return CSD_OK;
}

csd_status_t csd_ocm_reset(csd_ocm_t *ocm, void *stream)
{
    if (!ocm) return CSD_ERR_INVALID_ARG;
    chain_break();
    unsigned long long blocks = (ocm->n_slots + 255) / 256;
    const unsigned long long cap = static_cast<unsigned long long>(sm_count()) * 8;
    if (blocks > cap) blocks = cap;
    ocm_reset_kernel<<<static_cast<unsigned int>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        ocm->slots, ocm->n_slots, ocm->stats);
    return cudaGetLastError() == cudaSuccess ? CSD_OK : CSD_ERR_CUDA;
}

csd_status_t csd_ocm_destroy(csd_ocm_t *ocm)
{
    if (!ocm) return CSD_ERR_INVALID_ARG;
    chain_break();
    cudaError_t a = cudaFree(ocm->slots);
    cudaError_t b = cudaFree(ocm->stats);
    cudaError_t c = cudaFree(ocm->age_keys);
    cudaError_t d = cudaFree(ocm->age_counts);
    delete ocm;
    return (a == cudaSuccess && b == cudaSuccess && c == cudaSuccess && d == cudaSuccess) ? CSD_OK : CSD_ERR_CUDA;
}

csd_status_t csd_ocm_set_lambda(csd_ocm_t *ocm, uint32_t lambda)
{
    if (!ocm) return CSD_ERR_INVALID_ARG;
    ocm->lambda = lambda;
    return CSD_OK;
}

csd_status_t csd_ocm_set_shared(csd_ocm_t *ocm, int enable)
{
    if (!ocm) return CSD_ERR_INVALID_ARG;
    chain_break();
    if (ocm->shared && !enable) {
        // back to a single writer: the key count the ordered path starts from is brought up to date
        if (cudaDeviceSynchronize() != cudaSuccess ||
            cudaMemcpy(&ocm->stats->n_keys_start, &ocm->stats->n_keys, sizeof(unsigned long long), cudaMemcpyDeviceToDevice) != cudaSuccess) {
            (void)cudaGetLastError();
            return CSD_ERR_CUDA;
        }
    }
    ocm->shared = enable ? 1 : 0;
    return CSD_OK;
}

// ---- the step in two phases: batch rows that have stopped are not read any further ------------
namespace {
struct EarlyExitLayout {
    int first;                       // positions of the first phase
    size_t ws1, ws1_bytes, ws2, ws2_bytes, rows, n_alive, total;
};

bool early_exit_layout(int B, int K, int V, csd_dtype_t dtype, int first, EarlyExitLayout &l)
{
    if (!shape_ok(B, K, V, dtype) || K < 2) return false;
    if (first <= 0) first = (K + 1) / 3 > 1 ? (K + 1) / 3 : 1;
    if (first >= K) first = K - 1;
    l.first = first;
    Shape s1 = pick_shape(B, first, V, dtype, false);
    Shape s2 = pick_shape(B, K - first, V, dtype, false);
    s2.slots_per_row = s2.units_per_row < kListSlotsPerRow ? s2.units_per_row : kListSlotsPerRow;
    l.ws1 = 0;
    l.ws1_bytes = ws_layout(B, first, s1).total;
    l.ws2 = align_up(l.ws1_bytes, 256);
    l.ws2_bytes = ws_layout(B, K - first, s2).total;
    l.rows = align_up(l.ws2 + l.ws2_bytes, 256);
    l.n_alive = align_up(l.rows + static_cast<size_t>(B) * sizeof(int), 16);
    l.total = align_up(l.n_alive + 16, 256);
    return true;
}
}  // namespace

size_t csd_early_exit_workspace_bytes(int B, int K, int V, csd_dtype_t dtype, int first_phase_positions)
{
    EarlyExitLayout l;
    return early_exit_layout(B, K, V, dtype, first_phase_positions, l) ? l.total : 0;
}

csd_status_t csd_step_early_exit(const void *logits, csd_dtype_t dtype, int B, int K, int V, int64_t stride_b, int64_t stride_k,
                                 const int32_t *draft, csd_ocm_t *ocm, float tau, int first_phase_positions, int32_t *accept_len,
                                 int32_t *next_token, uint8_t *rescued_mask, int32_t *rej_draft, int32_t *rej_target,
                                 const csd_diag_t *diag, void *workspace, size_t workspace_bytes, void *stream)
{
    if (B <= 0 || K <= 0 || V <= 0 || (dtype != CSD_F32 && dtype != CSD_BF16)) return CSD_ERR_INVALID_ARG;
    if (K > CSD_MAX_K) return CSD_ERR_UNSUPPORTED;
    if (K < 2) return CSD_ERR_UNSUPPORTED;
    if (!workspace) return CSD_ERR_INVALID_ARG;
    EarlyExitLayout l;
    if (!early_exit_layout(B, K, V, dtype, first_phase_positions, l)) return CSD_ERR_UNSUPPORTED;
    if (workspace_bytes < l.total || (reinterpret_cast<uintptr_t>(workspace) & 15u)) return CSD_ERR_WORKSPACE;
    chain_break();
    char *ws = static_cast<char *>(workspace);
    int *rows = reinterpret_cast<int *>(ws + l.rows);
    int *n_alive = reinterpret_cast<int *>(ws + l.n_alive);
    PhaseSpec first = {K, 0, nullptr, nullptr, rows, n_alive, K, 1};
    csd_status_t rc = run_step(logits, dtype, B, l.first, V, stride_b, stride_k, draft, ocm, tau, accept_len, next_token, rescued_mask,
                               rej_draft, rej_target, diag, ws + l.ws1, l.ws1_bytes, stream, false, false, false, true, &first);
    if (rc != CSD_OK) return rc;
    PhaseSpec second = {K, l.first, rows, n_alive, nullptr, nullptr, 0, 0};
    rc = run_step(logits, dtype, B, K - l.first, V, stride_b, stride_k, draft, ocm, tau, accept_len, next_token, rescued_mask,
                  rej_draft, rej_target, diag, ws + l.ws2, l.ws2_bytes, stream, false, false, false, true, &second);
    if (rc != CSD_OK) return rc;
    return run_update(ocm, rej_draft, rej_target, nullptr, static_cast<int64_t>(B) * K, stream);
}

size_t csd_workspace_bytes(int B, int K, int V, csd_dtype_t dtype)
{
    if (!shape_ok(B, K, V, dtype)) return 0;
    // enough for either launch shape, so that csd_set_overlap does not change the answer
    const size_t a = ws_layout(B, K, pick_shape(B, K, V, dtype, false)).total;
    const size_t b = ws_layout(B, K, pick_shape(B, K, V, dtype, true)).total;
    return a > b ? a : b;
}

csd_status_t csd_workspace_init(void *workspace, size_t workspace_bytes, void *stream)
{
    if (!workspace || workspace_bytes == 0) return CSD_ERR_INVALID_ARG;
    chain_break();
    workspace_forget(workspace, workspace_bytes);
    if (cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return CSD_ERR_CUDA;
    }
    return CSD_OK;
}

csd_status_t csd_verify(const void *logits, csd_dtype_t dtype, int B, int K, int V, int64_t stride_b, int64_t stride_k,
                        const int32_t *draft, const csd_ocm_t *ocm, float tau, int32_t *accept_len, int32_t *next_token,
                        uint8_t *rescued_mask, int32_t *rej_draft, int32_t *rej_target, const csd_diag_t *diag,
                        void *workspace, size_t workspace_bytes, void *stream)
{
    return run_step(logits, dtype, B, K, V, stride_b, stride_k, draft, ocm, tau, accept_len, next_token, rescued_mask,
                    rej_draft, rej_target, diag, workspace, workspace_bytes, stream, false);
}

csd_status_t csd_step(const void *logits, csd_dtype_t dtype, int B, int K, int V, int64_t stride_b, int64_t stride_k,
                      const int32_t *draft, csd_ocm_t *ocm, float tau, int32_t *accept_len, int32_t *next_token,
                      uint8_t *rescued_mask, int32_t *rej_draft, int32_t *rej_target, const csd_diag_t *diag,
                      void *workspace, size_t workspace_bytes, void *stream)
{
    return run_step(logits, dtype, B, K, V, stride_b, stride_k, draft, ocm, tau, accept_len, next_token, rescued_mask,
                    rej_draft, rej_target, diag, workspace, workspace_bytes, stream, true);
}

csd_status_t csd_ocm_update(csd_ocm_t *ocm, const int32_t *rej_draft, const int32_t *rej_target, int64_t n, void *stream)
{
    return run_update(ocm, rej_draft, rej_target, nullptr, n, stream);
}

csd_status_t csd_ocm_import(csd_ocm_t *ocm, const int32_t *d, const int32_t *t, const uint32_t *cnt, uint64_t n,
                            void *stream)
{
    if (n > 0 && !cnt) return CSD_ERR_INVALID_ARG;
    if (n > (1ull << 62)) return CSD_ERR_INVALID_ARG;
    return run_update(ocm, d, t, cnt, static_cast<int64_t>(n), stream);
}

// staging layout of csd_step_host: logits | draft | accept_len | next_token | rescued |
// rej_draft | rej_target | workspace, each 256-byte aligned
namespace {
struct StagingLayout {
    size_t logits, draft, accept, next, rescued, rej_d, rej_t, ws, ws_bytes, total;
};
StagingLayout staging_layout(int B, int K, int V, csd_dtype_t dtype)
{
    StagingLayout s;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t at = off;
        off = align_up(off + bytes, 256);
        return at;
    };
    s.logits = take(static_cast<size_t>(B) * (K + 1) * V * elt_bytes(dtype));
    s.draft = take(static_cast<size_t>(B) * K * 4);
    s.accept = take(static_cast<size_t>(B) * 4);
    s.next = take(static_cast<size_t>(B) * 4);
    s.rescued = take(static_cast<size_t>(B) * K);
    s.rej_d = take(static_cast<size_t>(B) * K * 4);
    s.rej_t = take(static_cast<size_t>(B) * K * 4);
    s.ws_bytes = csd_workspace_bytes(B, K, V, dtype);
    s.ws = take(s.ws_bytes);
    s.total = off;
    return s;
}
}  // namespace

// ---- csd_verify_static: the verification step for callers that must not allocate ----------
//
// The scratch of the step kernel lives in this file-scope device array instead of a
// caller-provided workspace.  Every GPU that loads the library holds these bytes until the
// process exits.  In host code the array's name is only a host-side stand-in for the symbol;
// its device address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[CSD_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void *g_static_scratch_ptr[kMaxDevices];   // device address of g_static_scratch, per device
bool g_static_scratch_known[kMaxDevices];
std::mutex g_static_scratch_mutex;
}  // namespace

csd_status_t csd_verify_static(const void *logits, csd_dtype_t dtype, int B, int K, int V, int64_t stride_b,
                               int64_t stride_k, const int32_t *draft, const csd_ocm_t *ocm, float tau,
                               int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask, int32_t *rej_draft,
                               int32_t *rej_target, const csd_diag_t *diag, void *stream)
{
    if (!ocm) return CSD_ERR_INVALID_ARG;
    if (B <= 0 || K <= 0 || V <= 0 || (dtype != CSD_F32 && dtype != CSD_BF16)) return CSD_ERR_INVALID_ARG;
    if (K > CSD_MAX_K || !shape_ok(B, K, V, dtype)) return CSD_ERR_UNSUPPORTED;
    const size_t need = csd_workspace_bytes(B, K, V, dtype);
    if (need == 0 || need > CSD_STATIC_SCRATCH_BYTES) return CSD_ERR_WORKSPACE;   // shape needs more than the fixed scratch
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return CSD_ERR_CUDA;
    }
    if (dev != ocm->device) return CSD_ERR_INVALID_ARG;   // the memory's device must be the current one
    void *scratch = nullptr;
    {
        // once per device, with that device current (first call: not under stream capture); two host
        // threads may make their first call together
        std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
        if (!g_static_scratch_known[dev]) {
            void *ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
                (void)cudaGetLastError();
                return CSD_ERR_CUDA;
            }
            g_static_scratch_ptr[dev] = ptr;
            g_static_scratch_known[dev] = true;
        }
        scratch = g_static_scratch_ptr[dev];
    }
    // The array keeps whatever the last call (possibly of another shape) left in it, and the
    // kernel needs its counters and sequence words to start at zero: clear the part in use.
    if (cudaMemsetAsync(scratch, 0, need, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return CSD_ERR_CUDA;
    }
    return run_step(logits, dtype, B, K, V, stride_b, stride_k, draft, ocm, tau, accept_len, next_token, rescued_mask,
                    rej_draft, rej_target, diag, scratch, need, stream, false, /*may_chain=*/false,
                    /*may_overlap=*/false, /*track_layout=*/false);   // cleared just above, whatever it held
}

// ---- the step taken straight from the LM head --------------------------------------------------
namespace {

struct LmheadPlan {
    bool pair;              // CTA pairs (clusters of two) instead of lone CTAs
    int grid, n_tile, tiles_total, tiles_per_cta;
    int rows1, rows2, a_bytes, sub_bytes, kps, n_stages, smem_bytes;
    size_t partials_off, zd_off, total;
};

bool lmhead_shape_ok(int B, int K, int H, int V)
{
    if (!(B > 0 && K > 0 && K <= CSD_MAX_K && V > 0 && H > 0)) return false;
    if (H % lmhead::kBlockK != 0) return false;
    return static_cast<long long>(B) * (K + 1) <= (1ll << 20) && static_cast<long long>(V) < (1ll << 30);
}

int g_lmhead_kblocks_per_stage = 0;   // 0 = automatic
int g_lmhead_pairing = 0;             // 0 = automatic, 1 = lone CTAs, 2 = CTA pairs
int g_lmhead_tile_cols = 0;           // 0 = automatic; else the columns of one MMA (a multiple of 16, 16..256)
int g_lmhead_wide_fetch = 1;          // W rows come into L2 256 bytes at a time (two consecutive k-blocks of a row)

void lmhead_place_workspace(LmheadPlan &pl, size_t rows, int B, int K)
{
    pl.partials_off = 0;
    pl.zd_off = align_up(rows * pl.grid * sizeof(Partial), 256);
    pl.total = align_up(pl.zd_off + static_cast<size_t>(B) * K * sizeof(float), 256);
}

// Lone CTAs: the vocabulary is cut into tiles of n_tile columns (a multiple of 16, at most 256) such that every CTA of
// a one-per-SM grid owns the same number of consecutive tiles.
LmheadPlan lmhead_plan_lone(int B, int K, int H, int V)
{
    LmheadPlan pl;
    pl.pair = false;
    const long long sms = sm_count();
    long long per = (V + sms * lmhead::kNMax - 1) / (sms * lmhead::kNMax);          // tiles per CTA
    if (per < 1) per = 1;
    long long width = (V + sms * per - 1) / (sms * per);
    width = (width + 15) / 16 * 16;
    if (width > lmhead::kNMax) width = lmhead::kNMax;
    if (width < 16) width = 16;
    if (g_lmhead_tile_cols > 0) {
        width = g_lmhead_tile_cols;
        per = (V + sms * width - 1) / (sms * width);
    }
    pl.n_tile = static_cast<int>(width);
    pl.tiles_total = static_cast<int>((V + width - 1) / width);
    pl.tiles_per_cta = static_cast<int>(per);
    long long grid = (pl.tiles_total + per - 1) / per;
    pl.grid = static_cast<int>(grid < 1 ? 1 : grid);
    const size_t rows = static_cast<size_t>(B) * (K + 1);
    // shared-memory ring: as many stages as fit beside the barriers, the alignment room and the slack
    const size_t groups = (rows + lmhead::kRowsMax - 1) / lmhead::kRowsMax;
    const size_t rows_last = rows - (groups - 1) * lmhead::kRowsMax;
    pl.rows2 = rows_last > lmhead::kMTile ? static_cast<int>((rows_last - lmhead::kMTile + 7) / 8 * 8) : 0;
    pl.rows1 = rows_last >= lmhead::kMTile ? lmhead::kMTile : static_cast<int>((rows_last + 7) / 8 * 8);
    const int rows2_most = groups > 1 ? lmhead::kMTile : pl.rows2;
    const int rows1_most = groups > 1 ? lmhead::kMTile : pl.rows1;           // a lone short group: W follows its rows at once
    pl.a_bytes = static_cast<int>(align_up(static_cast<size_t>(rows1_most + rows2_most) * lmhead::kRowBytes, 1024));
    pl.sub_bytes = pl.a_bytes + static_cast<int>(align_up(static_cast<size_t>(pl.n_tile) * lmhead::kRowBytes, 1024));
    const int fixed = 1024 + lmhead::kBarrierBytes + lmhead::kSlackBytes;
    pl.kps = g_lmhead_kblocks_per_stage > 0 ? g_lmhead_kblocks_per_stage : 1;
    while (pl.kps > 1 && (H % (lmhead::kBlockK * pl.kps) != 0 || (lmhead::kSmemLimit - fixed) / (pl.kps * pl.sub_bytes) < 2)) --pl.kps;
    int stages = (lmhead::kSmemLimit - fixed) / (pl.kps * pl.sub_bytes);
    pl.n_stages = stages > lmhead::kMaxStages ? lmhead::kMaxStages : stages;
    pl.smem_bytes = fixed + pl.n_stages * pl.kps * pl.sub_bytes;
    lmhead_place_workspace(pl, rows, B, K);
    return pl;
}

// CTA pairs: a pair's tile has 2 n_tile columns (n_tile a multiple of 16, at most 256), every pair of a one-CTA-per-SM
// grid owns the same number of consecutive tiles; each CTA holds half of a row group's rows.
LmheadPlan lmhead_plan_pair(int B, int K, int /*H*/, int V)
{
    LmheadPlan pl;
    pl.pair = true;
    const long long pairs = sm_count() / 2;
    const long long widest = 2 * lmhead::kNMax;
    long long per = (V + pairs * widest - 1) / (pairs * widest);                    // tiles per pair
    if (per < 1) per = 1;
    long long width = (V + pairs * per - 1) / (pairs * per);                        // columns of a pair's tile
    long long n = ((width + 1) / 2 + 15) / 16 * 16;
    if (n > lmhead::kNMax) n = lmhead::kNMax;
    if (n < 16) n = 16;
    if (g_lmhead_tile_cols > 0) {
        n = g_lmhead_tile_cols;
        per = (V + pairs * 2 * n - 1) / (pairs * 2 * n);
    }
    pl.n_tile = static_cast<int>(n);
    pl.tiles_total = static_cast<int>((V + 2 * n - 1) / (2 * n));
    pl.tiles_per_cta = static_cast<int>(per);
    long long used = (pl.tiles_total + per - 1) / per;
    pl.grid = static_cast<int>(2 * (used < 1 ? 1 : used));
    const size_t rows = static_cast<size_t>(B) * (K + 1);
    const size_t groups = (rows + lmhead::kRowsMax - 1) / lmhead::kRowsMax;
    const size_t rows_last = rows - (groups - 1) * lmhead::kRowsMax;
    pl.rows2 = static_cast<int>(((rows_last + 1) / 2 + 7) / 8 * 8);                 // rows per CTA in the last group
    pl.rows1 = pl.rows2;
    const int half_most = groups > 1 ? lmhead::kMTile : pl.rows2;
    pl.a_bytes = half_most * lmhead::kRowBytes;                                      // a multiple of 1 KiB: 8 rows
    pl.sub_bytes = pl.a_bytes + pl.n_tile * lmhead::kRowBytes;                       // + two sub-tiles of n_tile / 2 rows
    const int fixed = 1024 + lmhead::kBarrierBytes + lmhead::kSlackBytes;
    pl.kps = 1;
    int stages = (lmhead::kSmemLimit - fixed) / pl.sub_bytes;
    pl.n_stages = stages > lmhead::kMaxStages ? lmhead::kMaxStages : stages;
    pl.smem_bytes = fixed + pl.n_stages * pl.sub_bytes;
    lmhead_place_workspace(pl, rows, B, K);
    return pl;
}

// Once per device: lets both GEMM kernels use the shared memory they need and asks whether the device can hold a
// cluster of two such blocks at all (it cannot in some partitioned configurations).  -1: a CUDA call failed;
// 0: no device in this process (planning only); 1: one-CTA kernel only; 2: pairs possible.
int lmhead_device_state()
{
    static std::mutex m;
    static int state[kMaxLmheadDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    if (dev < 0 || dev >= kMaxLmheadDevices) return -1;
    std::lock_guard<std::mutex> lock(m);
    if (state[dev] == 0) {
        if (cudaFuncSetAttribute(lmhead::lmhead_stats_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, lmhead::kSmemLimit) !=
                cudaSuccess ||
            cudaFuncSetAttribute(lmhead::lmhead_stats_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 lmhead::kSmemLimit) != cudaSuccess) {
            (void)cudaGetLastError();
            return -1;
        }
        cudaLaunchConfig_t probe;
        std::memset(&probe, 0, sizeof probe);
        probe.gridDim = dim3(2);
        probe.blockDim = dim3(lmhead::kThreads);
        probe.dynamicSmemBytes = static_cast<size_t>(lmhead::kSmemLimit);
        cudaLaunchAttribute cl[1];
        cl[0].id = cudaLaunchAttributeClusterDimension;
        cl[0].val.clusterDim.x = 2;
        cl[0].val.clusterDim.y = 1;
        cl[0].val.clusterDim.z = 1;
        probe.attrs = cl;
        probe.numAttrs = 1;
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, lmhead::lmhead_stats_pair_kernel, &probe) != cudaSuccess) {
            (void)cudaGetLastError();
            clusters = 0;
        }
        state[dev] = clusters >= 1 ? 2 : 1;
    }
    return state[dev];
}

// Pairs pay when the hidden rows are a large part of what a k-block brings into shared memory.
bool lmhead_wants_pair(int B, int K)
{
    if (sm_count() < 2) return false;
    const int dev_state = lmhead_device_state();
    if (dev_state == 1 || dev_state < 0) return false;
    if (g_lmhead_pairing == 1) return false;
    if (g_lmhead_pairing == 2) return true;
    return static_cast<long long>(B) * (K + 1) > lmhead::kMTile;
}

LmheadPlan lmhead_plan(int B, int K, int H, int V)
{
    return lmhead_wants_pair(B, K) ? lmhead_plan_pair(B, K, H, V) : lmhead_plan_lone(B, K, H, V);
}

// What a workspace must hold whichever kernel runs.
size_t lmhead_workspace_most(int B, int K, int H, int V)
{
    const size_t a = lmhead_plan_lone(B, K, H, V).total;
    const size_t b = sm_count() >= 2 ? lmhead_plan_pair(B, K, H, V).total : 0;
    return a > b ? a : b;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static std::mutex m;
    static EncodeTiledFn fn = nullptr;
    std::lock_guard<std::mutex> lock(m);
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &res) != cudaSuccess ||
            res != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// A [rows, cols] row-major bf16 matrix as a tensor map whose box is box_rows x 64 columns, 128-byte swizzle;
// elements outside the matrix read as zero.
bool make_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, bool wide_fetch = false)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(lmhead::kBlockK), box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              wide_fetch ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

csd_status_t run_lmhead(const void *hidden, const void *weight, int B, int K, int H, int V, const int32_t *draft, csd_ocm *ocm,
                        float tau, int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask, int32_t *rej_draft,
                        int32_t *rej_target, const csd_diag_t *diag, void *workspace, size_t workspace_bytes, void *stream,
                        bool do_update)
{
    if (!hidden || !weight || !draft || !ocm || !accept_len || !next_token || !rescued_mask || !rej_draft || !rej_target || !workspace)
        return CSD_ERR_INVALID_ARG;
    if (B <= 0 || K <= 0 || H <= 0 || V <= 0) return CSD_ERR_INVALID_ARG;
    if (!(tau >= 0.0f) || std::isinf(tau)) return CSD_ERR_INVALID_ARG;
    if (!lmhead_shape_ok(B, K, H, V)) return CSD_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(hidden) & 15u) || (reinterpret_cast<uintptr_t>(weight) & 15u)) return CSD_ERR_INVALID_ARG;
    const LmheadPlan pl = lmhead_plan(B, K, H, V);
    if (workspace_bytes < lmhead_workspace_most(B, K, H, V) || (reinterpret_cast<uintptr_t>(workspace) & 15u)) return CSD_ERR_WORKSPACE;
    chain_break();
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int R = B * (K + 1);

    if (lmhead_device_state() < 0) return CSD_ERR_CUDA;
    CUtensorMap map_h, map_h2, map_w;
    if (!make_map(&map_h, hidden, static_cast<uint64_t>(R), static_cast<uint64_t>(H), lmhead::kMTile) ||
        !make_map(&map_h2, hidden, static_cast<uint64_t>(R), static_cast<uint64_t>(H),
                  static_cast<uint32_t>(pl.rows2 ? pl.rows2 : pl.rows1)) ||
        !make_map(&map_w, weight, static_cast<uint64_t>(V), static_cast<uint64_t>(H),
                  static_cast<uint32_t>(pl.pair ? pl.n_tile / 2 : pl.n_tile), g_lmhead_wide_fetch != 0))
        return CSD_ERR_CUDA;

    char *ws = static_cast<char *>(workspace);
    lmhead::Params p;
    std::memset(&p, 0, sizeof p);
    p.R = R; p.H = H; p.V = V; p.B = B; p.K = K;
    p.n_tile = pl.n_tile;
    p.tiles_total = pl.tiles_total;
    p.tiles_per_cta = pl.tiles_per_cta;
    p.rows1 = pl.rows1;
    p.rows2 = pl.rows2;
    p.a_bytes = pl.a_bytes;
    p.sub_bytes = pl.sub_bytes;
    p.kblocks_per_stage = pl.kps;
    p.n_stages = pl.n_stages;
    p.draft = draft;
    p.partials = reinterpret_cast<Partial *>(ws + pl.partials_off);
    p.zd = reinterpret_cast<float *>(ws + pl.zd_off);
    p.stats = ocm->stats;
    {
        // With step overlap on, launched programmatically: behind this library's own update kernel (which lets its
        // dependents in at once) the GEMM of this step streams W while the decisions and the update of the step before
        // finish; it waits for them before its first store.  It reads its inputs before that wait, hence the opt-in.
        cudaLaunchConfig_t cfg;
        std::memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3(static_cast<unsigned int>(pl.grid));
        cfg.blockDim = dim3(lmhead::kThreads);
        cfg.dynamicSmemBytes = static_cast<size_t>(pl.smem_bytes);
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = 2;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        // (not for pairs: measured, a cluster grid that comes in beside the tail of the step before is slower, 257 us
        // per step against 248 at 192 rows, where the one-CTA kernel gains 20 us at 9 rows)
        const bool early = g_overlap_steps != 0 && !pl.pair;
        if (!early) attr[0] = attr[1];
        cfg.attrs = attr;
        cfg.numAttrs = (early ? 1 : 0) + (pl.pair ? 1 : 0);
        const cudaError_t err = pl.pair ? cudaLaunchKernelEx(&cfg, lmhead::lmhead_stats_pair_kernel, map_h, map_h2, map_w, p)
                                        : cudaLaunchKernelEx(&cfg, lmhead::lmhead_stats_kernel, map_h, map_h2, map_w, p);
        if (err != cudaSuccess) {
            (void)cudaGetLastError();
            return CSD_ERR_CUDA;
        }
    }

    lmhead::FinalizeParams f;
    std::memset(&f, 0, sizeof f);
    f.B = B; f.K = K; f.V = V; f.n_parts = pl.grid;
    f.partials = p.partials;
    f.zd = p.zd;
    f.draft = draft;
    f.ocm = view_of(ocm);
    f.log_tau = csd_scg_threshold(tau);
    f.accept_len = accept_len; f.next_token = next_token; f.rescued = rescued_mask;
    f.rej_d = rej_draft; f.rej_t = rej_target;
    if (diag) f.diag = *diag;
    {
        cudaLaunchConfig_t cfg;
        std::memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3(static_cast<unsigned int>(B));
        cfg.blockDim = dim3(32 * lmhead::kFinalizeWarps);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, lmhead::lmhead_finalize_kernel, f) != cudaSuccess) {
            (void)cudaGetLastError();
            return CSD_ERR_CUDA;
        }
    }
    if (do_update) return run_update(ocm, rej_draft, rej_target, nullptr, static_cast<int64_t>(B) * K, stream, true);
    return CSD_OK;
}

}  // namespace

size_t csd_lmhead_workspace_bytes(int B, int K, int H, int V)
{
    if (!lmhead_shape_ok(B, K, H, V)) return 0;
    return lmhead_workspace_most(B, K, H, V);
}

csd_status_t csd_verify_lmhead(const void *hidden, const void *weight, int B, int K, int H, int V, const int32_t *draft,
                               const csd_ocm_t *ocm, float tau, int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask,
                               int32_t *rej_draft, int32_t *rej_target, const csd_diag_t *diag, void *workspace,
                               size_t workspace_bytes, void *stream)
{
    return run_lmhead(hidden, weight, B, K, H, V, draft, const_cast<csd_ocm_t *>(ocm), tau, accept_len, next_token, rescued_mask,
                      rej_draft, rej_target, diag, workspace, workspace_bytes, stream, false);
}

csd_status_t csd_step_lmhead(const void *hidden, const void *weight, int B, int K, int H, int V, const int32_t *draft, csd_ocm_t *ocm,
                             float tau, int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask, int32_t *rej_draft,
                             int32_t *rej_target, const csd_diag_t *diag, void *workspace, size_t workspace_bytes, void *stream)
{
    return run_lmhead(hidden, weight, B, K, H, V, draft, ocm, tau, accept_len, next_token, rescued_mask, rej_draft, rej_target,
                      diag, workspace, workspace_bytes, stream, true);
}

csd_status_t csd_lmhead_set_tuning(int kblocks_per_stage, int mma_cols)
{
    if (kblocks_per_stage < 0 || kblocks_per_stage > 4) return CSD_ERR_INVALID_ARG;
    if (mma_cols != 0 && (mma_cols < 16 || mma_cols > lmhead::kNMax || mma_cols % 16 != 0)) return CSD_ERR_INVALID_ARG;
    g_lmhead_kblocks_per_stage = kblocks_per_stage;
    g_lmhead_tile_cols = mma_cols;
    return CSD_OK;
}

csd_status_t csd_sampled_set_rounds(int mode)
{
    if (mode < 0 || mode > 2) return CSD_ERR_INVALID_ARG;
    g_sampled_rounds = mode;
    return CSD_OK;
}

int csd_sampled_launches(int B, int K, int V, csd_dtype_t dtype)
{
    if (!shape_ok(B, K, V, dtype)) return 0;
    return sampled_single_round(B, K, V, dtype == CSD_BF16 ? 2 : 4) ? 5 : 7;
}

csd_status_t csd_lmhead_set_pairing(int mode)
{
    if (mode < 0 || mode > 2) return CSD_ERR_INVALID_ARG;
    g_lmhead_pairing = mode;
    return CSD_OK;
}

int csd_lmhead_uses_pairs(int B, int K)
{
    return (B > 0 && K > 0 && lmhead_wants_pair(B, K)) ? 1 : 0;
}

csd_status_t csd_lmhead_shape(int B, int K, int H, int V, int *grid, int *tile_cols, int *tiles, int *tiles_per_block)
{
    if (!lmhead_shape_ok(B, K, H, V)) return CSD_ERR_UNSUPPORTED;
    const LmheadPlan pl = lmhead_plan(B, K, H, V);
    if (grid) *grid = pl.grid;
    if (tile_cols) *tile_cols = pl.pair ? 2 * pl.n_tile : pl.n_tile;
    if (tiles) *tiles = pl.tiles_total;
    if (tiles_per_block) *tiles_per_block = pl.tiles_per_cta;
    return CSD_OK;
}

size_t csd_sampled_workspace_bytes(int B, int K, int V, csd_dtype_t dtype)
{
    if (!shape_ok(B, K, V, dtype)) return 0;
    return sampled_layout(B, K, V).total;
}

csd_status_t csd_verify_sampled(const void *logits, const void *draft_logits, csd_dtype_t dtype, int B, int K, int V,
                                int64_t stride_b, int64_t stride_k, int64_t draft_stride_b, int64_t draft_stride_k,
                                const int32_t *draft, const float *r_accept, uint64_t seed, float temperature,
                                const csd_ocm_t *ocm, float tau, int32_t *accept_len, int32_t *next_token,
                                uint8_t *rescued_mask, int32_t *rej_draft, int32_t *rej_target,
                                const csd_sampled_diag_t *diag, void *workspace, size_t workspace_bytes, void *stream)
{
    return run_sampled(logits, draft_logits, dtype, B, K, V, stride_b, stride_k, draft_stride_b, draft_stride_k, draft,
                       r_accept, seed, temperature, const_cast<csd_ocm_t *>(ocm), tau, accept_len, next_token,
                       rescued_mask, rej_draft, rej_target, diag, workspace, workspace_bytes, stream, false);
}

csd_status_t csd_step_sampled(const void *logits, const void *draft_logits, csd_dtype_t dtype, int B, int K, int V,
                              int64_t stride_b, int64_t stride_k, int64_t draft_stride_b, int64_t draft_stride_k,
                              const int32_t *draft, const float *r_accept, uint64_t seed, float temperature,
                              csd_ocm_t *ocm, float tau, int32_t *accept_len, int32_t *next_token,
                              uint8_t *rescued_mask, int32_t *rej_draft, int32_t *rej_target,
                              const csd_sampled_diag_t *diag, void *workspace, size_t workspace_bytes, void *stream)
{
    return run_sampled(logits, draft_logits, dtype, B, K, V, stride_b, stride_k, draft_stride_b, draft_stride_k, draft,
                       r_accept, seed, temperature, ocm, tau, accept_len, next_token, rescued_mask, rej_draft,
                       rej_target, diag, workspace, workspace_bytes, stream, true);
}

size_t csd_host_staging_bytes(int B, int K, int V, csd_dtype_t dtype)
{
    if (!shape_ok(B, K, V, dtype)) return 0;
    return staging_layout(B, K, V, dtype).total;
}

csd_status_t csd_step_host(const void *logits_host, csd_dtype_t dtype, int B, int K, int V, const int32_t *draft_host,
                           csd_ocm_t *ocm, float tau, int32_t *accept_len_host, int32_t *next_token_host,
                           uint8_t *rescued_mask_host, void *staging, size_t staging_bytes, void *stream)
{
    if (!logits_host || !draft_host || !ocm || !accept_len_host || !next_token_host || !rescued_mask_host || !staging)
        return CSD_ERR_INVALID_ARG;
    if (B <= 0 || K <= 0 || V <= 0 || (dtype != CSD_F32 && dtype != CSD_BF16)) return CSD_ERR_INVALID_ARG;
    if (K > CSD_MAX_K || !shape_ok(B, K, V, dtype)) return CSD_ERR_UNSUPPORTED;
    const StagingLayout s = staging_layout(B, K, V, dtype);
    if (staging_bytes < s.total || (reinterpret_cast<uintptr_t>(staging) & 255u)) return CSD_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char *dev = static_cast<char *>(staging);
    chain_break();   // the workspace inside the staging area is cleared below
    const size_t lbytes = static_cast<size_t>(B) * (K + 1) * V * elt_bytes(dtype);
    bool ok = true;
    ok = ok && cudaMemcpyAsync(dev + s.logits, logits_host, lbytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(dev + s.draft, draft_host, static_cast<size_t>(B) * K * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    // the arrival counters sit at the end of the workspace; clearing it all keeps the staging stateless
    ok = ok && cudaMemsetAsync(dev + s.ws, 0, s.ws_bytes, st) == cudaSuccess;
    if (!ok) {
        (void)cudaGetLastError();
        return CSD_ERR_CUDA;
    }
    const csd_status_t rc =
        run_step(dev + s.logits, dtype, B, K, V, static_cast<int64_t>(K + 1) * V, V,
                 reinterpret_cast<const int32_t *>(dev + s.draft), ocm, tau, reinterpret_cast<int32_t *>(dev + s.accept),
                 reinterpret_cast<int32_t *>(dev + s.next), reinterpret_cast<uint8_t *>(dev + s.rescued),
                 reinterpret_cast<int32_t *>(dev + s.rej_d), reinterpret_cast<int32_t *>(dev + s.rej_t), nullptr,
                 dev + s.ws, s.ws_bytes, stream, /*do_update=*/true, /*may_chain=*/true,
                 /*may_overlap=*/true, /*track_layout=*/false);
    if (rc != CSD_OK) return rc;
    ok = ok && cudaMemcpyAsync(accept_len_host, dev + s.accept, static_cast<size_t>(B) * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(next_token_host, dev + s.next, static_cast<size_t>(B) * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(rescued_mask_host, dev + s.rescued, static_cast<size_t>(B) * K, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
    if (!ok) {
        (void)cudaGetLastError();
        return CSD_ERR_CUDA;
    }
    return CSD_OK;
}

csd_status_t csd_ocm_export(const csd_ocm_t *ocm, int32_t *d, int32_t *t, uint32_t *cnt, uint64_t cap, uint64_t *n_out,
                            void *stream)
{
    if (!ocm || !n_out || (cap > 0 && (!d || !t || !cnt))) return CSD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    bool ok = cudaMemsetAsync(&ocm->stats->export_count, 0, sizeof(unsigned long long), st) == cudaSuccess;
    if (ok) {
        unsigned long long blocks = (ocm->n_slots + 255) / 256;
        const unsigned long long capb = static_cast<unsigned long long>(sm_count()) * 8;
        if (blocks > capb) blocks = capb;
        ocm_export_kernel<<<static_cast<unsigned int>(blocks), 256, 0, st>>>(view_of(ocm), d, t, cnt, cap);
        ok = cudaGetLastError() == cudaSuccess;
    }
    unsigned long long n = 0;
    ok = ok && cudaMemcpyAsync(&n, &ocm->stats->export_count, sizeof n, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
    if (!ok) {
        (void)cudaGetLastError();
        return CSD_ERR_CUDA;
    }
    *n_out = n;
    return CSD_OK;
}

csd_status_t csd_ocm_age(csd_ocm_t *ocm, void *stream)
{
    if (!ocm) return CSD_ERR_INVALID_ARG;
    chain_break();
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(&ocm->stats->export_count, 0, sizeof(unsigned long long), st) != cudaSuccess) {
        (void)cudaGetLastError();
        return CSD_ERR_CUDA;
    }
    unsigned long long blocks = (ocm->n_slots + 255) / 256;
    const unsigned long long cap = static_cast<unsigned long long>(sm_count()) * 8;
    if (blocks > cap) blocks = cap;
    ocm_age_collect_kernel<<<static_cast<unsigned int>(blocks), 256, 0, st>>>(view_of(ocm), ocm->age_keys, ocm->age_counts);
    if (cudaGetLastError() != cudaSuccess) return CSD_ERR_CUDA;
    unsigned long long blocks2 = (ocm->n_slots / 2 + 255) / 256;
    if (blocks2 > cap) blocks2 = cap;
    ocm_age_reinsert_kernel<<<static_cast<unsigned int>(blocks2), 256, 0, st>>>(view_of(ocm), ocm->age_keys, ocm->age_counts);
    return cudaGetLastError() == cudaSuccess ? CSD_OK : CSD_ERR_CUDA;
}

// ---- the memory as sorted triples on the host: file format and merge ------------------------
namespace {

struct Triple {
    int32_t d, t;
    uint32_t c;
};

// Every stored pair, sorted by (draft, target).  Synchronises `stream`.
csd_status_t sorted_triples(const csd_ocm *ocm, std::vector<Triple> &out, cudaStream_t st)
{
    out.clear();
    const uint64_t cap = ocm->n_slots / 2;
    int32_t *dd = nullptr, *dt = nullptr;
    uint32_t *dc = nullptr;
    if (cudaMalloc(&dd, cap * 4) != cudaSuccess || cudaMalloc(&dt, cap * 4) != cudaSuccess || cudaMalloc(&dc, cap * 4) != cudaSuccess) {
        (void)cudaGetLastError();
        cudaFree(dd); cudaFree(dt); cudaFree(dc);
        (void)cudaGetLastError();
        return CSD_ERR_OOM;
    }
    uint64_t n = 0;
    csd_status_t rc = csd_ocm_export(ocm, dd, dt, dc, cap, &n, st);
    if (rc == CSD_OK) {
        if (n > cap) n = cap;
        std::vector<int32_t> hd(n), ht(n);
        std::vector<uint32_t> hc(n);
        bool ok = true;
        if (n) {
            ok = cudaMemcpyAsync(hd.data(), dd, n * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess &&
                 cudaMemcpyAsync(ht.data(), dt, n * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess &&
                 cudaMemcpyAsync(hc.data(), dc, n * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess &&
                 cudaStreamSynchronize(st) == cudaSuccess;
        }
        if (!ok) {
            (void)cudaGetLastError();
            rc = CSD_ERR_CUDA;
        } else {
            out.resize(n);
            for (uint64_t j = 0; j < n; ++j) out[j] = Triple{hd[j], ht[j], hc[j]};
            std::sort(out.begin(), out.end(), [](const Triple &a, const Triple &b) { return a.d != b.d ? a.d < b.d : a.t < b.t; });
        }
    }
    cudaFree(dd); cudaFree(dt); cudaFree(dc);
    return rc;
}

// count[(d, t)] += c for the triples in order.  Synchronises `stream`.
csd_status_t add_triples(csd_ocm *ocm, const std::vector<Triple> &tr, cudaStream_t st)
{
    const size_t n = tr.size();
    if (n == 0) return CSD_OK;
    std::vector<int32_t> hd(n), ht(n);
    std::vector<uint32_t> hc(n);
    for (size_t j = 0; j < n; ++j) { hd[j] = tr[j].d; ht[j] = tr[j].t; hc[j] = tr[j].c; }
    int32_t *dd = nullptr, *dt = nullptr;
    uint32_t *dc = nullptr;
    if (cudaMalloc(&dd, n * 4) != cudaSuccess || cudaMalloc(&dt, n * 4) != cudaSuccess || cudaMalloc(&dc, n * 4) != cudaSuccess) {
        (void)cudaGetLastError();
        cudaFree(dd); cudaFree(dt); cudaFree(dc);
        (void)cudaGetLastError();
        return CSD_ERR_OOM;
    }
    csd_status_t rc = CSD_OK;
    if (cudaMemcpyAsync(dd, hd.data(), n * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(dt, ht.data(), n * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(dc, hc.data(), n * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        (void)cudaGetLastError();
        rc = CSD_ERR_CUDA;
    }
    if (rc == CSD_OK) rc = csd_ocm_import(ocm, dd, dt, dc, n, st);
    if (cudaStreamSynchronize(st) != cudaSuccess) {
        (void)cudaGetLastError();
        rc = rc == CSD_OK ? CSD_ERR_CUDA : rc;
    }
    cudaFree(dd); cudaFree(dt); cudaFree(dc);
    return rc;
}

constexpr char kFileMagic[8] = {'C', 'S', 'D', 'O', 'C', 'M', '\0', '\0'};
constexpr uint32_t kFileVersion = 1;

struct FileHeader {            // 64 bytes, little-endian, see csd.h
    char magic[8];
    uint32_t version, lambda;
    uint64_t n_slots, n, n_dropped;
    uint8_t reserved[24];
};
static_assert(sizeof(FileHeader) == 64, "file header layout");
static_assert(sizeof(Triple) == 12, "file record layout");

}  // namespace

csd_status_t csd_ocm_merge(csd_ocm_t *dst, const csd_ocm_t *src, void *stream)
{
    if (!dst || !src || dst == src) return CSD_ERR_INVALID_ARG;
    if (dst->device != src->device) return CSD_ERR_UNSUPPORTED;
    std::vector<Triple> tr;
    const csd_status_t rc = sorted_triples(src, tr, static_cast<cudaStream_t>(stream));
    if (rc != CSD_OK) return rc;
    return add_triples(dst, tr, static_cast<cudaStream_t>(stream));
}

csd_status_t csd_ocm_save(const csd_ocm_t *ocm, const char *path, void *stream)
{
    if (!ocm || !path) return CSD_ERR_INVALID_ARG;
    std::vector<Triple> tr;
    csd_status_t rc = sorted_triples(ocm, tr, static_cast<cudaStream_t>(stream));
    if (rc != CSD_OK) return rc;
    csd_stats_t st;
    rc = csd_ocm_stats(ocm, &st, stream);
    if (rc != CSD_OK) return rc;
    FileHeader h;
    std::memset(&h, 0, sizeof h);
    std::memcpy(h.magic, kFileMagic, 8);
    h.version = kFileVersion;
    h.lambda = ocm->lambda;
    h.n_slots = ocm->n_slots;
    h.n = tr.size();
    h.n_dropped = st.n_dropped;
    FILE *f = std::fopen(path, "wb");
    if (!f) return CSD_ERR_IO;
    bool ok = std::fwrite(&h, sizeof h, 1, f) == 1;
    if (ok && !tr.empty()) ok = std::fwrite(tr.data(), sizeof(Triple), tr.size(), f) == tr.size();
    ok = (std::fclose(f) == 0) && ok;
    return ok ? CSD_OK : CSD_ERR_IO;
}

csd_status_t csd_ocm_load(csd_ocm_t **out, const char *path, uint64_t n_slots, int device)
{
    if (!out || !path) return CSD_ERR_INVALID_ARG;
    *out = nullptr;
    FILE *f = std::fopen(path, "rb");
    if (!f) return CSD_ERR_IO;
    FileHeader h;
    std::vector<Triple> tr;
    bool ok = std::fread(&h, sizeof h, 1, f) == 1 && std::memcmp(h.magic, kFileMagic, 8) == 0 && h.version == kFileVersion &&
              h.n <= (1ull << 29);
    if (ok) {
        tr.resize(h.n);
        if (h.n) ok = std::fread(tr.data(), sizeof(Triple), h.n, f) == h.n;
    }
    std::fclose(f);
    if (!ok) return CSD_ERR_IO;
    for (size_t j = 0; j < tr.size(); ++j) {      // a well-formed file: valid pairs, strictly ascending
        if (tr[j].d < 0 || tr[j].t < 0) return CSD_ERR_IO;
        if (j && !(tr[j - 1].d < tr[j].d || (tr[j - 1].d == tr[j].d && tr[j - 1].t < tr[j].t))) return CSD_ERR_IO;
    }
    csd_ocm_t *o = nullptr;
    csd_status_t rc = csd_ocm_create(&o, n_slots ? n_slots : h.n_slots, h.lambda, device);
    if (rc != CSD_OK) return rc;
    rc = add_triples(o, tr, nullptr);
    if (rc != CSD_OK) {
        csd_ocm_destroy(o);
        return rc;
    }
    *out = o;
    return CSD_OK;
}

csd_status_t csd_ocm_stats(const csd_ocm_t *ocm, csd_stats_t *host_out, void *stream)
{
    if (!ocm || !host_out) return CSD_ERR_INVALID_ARG;
    OcmStatsDev s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&s, ocm->stats, sizeof s, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        (void)cudaGetLastError();
        return CSD_ERR_CUDA;
    }
    host_out->n_slots = ocm->n_slots;
    host_out->key_limit = ocm->n_slots / 2;
    host_out->n_keys = s.n_keys;
    host_out->n_dropped = s.n_dropped;
    host_out->steps = s.steps;
    host_out->positions = s.positions;
    host_out->matches = s.matches;
    host_out->rescues = s.rescues;
    host_out->rejections = s.rejections;
    host_out->lambda = ocm->lambda;
    host_out->flags = s.flags;
    host_out->debug_site = s.debug_site;
    host_out->reserved = 0;
    return CSD_OK;
}

float csd_scg_threshold(float tau)
{
    if (tau == 0.0f) return -INFINITY;
    return static_cast<float>(std::log(static_cast<double>(tau)));
}

csd_status_t csd_launch_shape(int B, int K, int V, csd_dtype_t dtype, int *grid, int *block, int *chunk_elems,
                              int *parts_per_row)
{
    if (!shape_ok(B, K, V, dtype)) return CSD_ERR_INVALID_ARG;
    const Shape s = pick_shape(B, K, V, dtype, g_overlap_steps != 0);
    if (grid) *grid = s.grid;
    if (block) *block = s.block;
    if (chunk_elems) *chunk_elems = s.chunk_units * s.unit_elems;
    if (parts_per_row) *parts_per_row = s.slots_per_row;
    return CSD_OK;
}

csd_status_t csd_set_tuning(int chunk_bytes, int ctas_per_sm, int block_threads)
{
    if (chunk_bytes != 0 && (chunk_bytes < 512 || chunk_bytes % 512 != 0 || chunk_bytes > (1 << 22))) return CSD_ERR_INVALID_ARG;
    if (ctas_per_sm < 0 || ctas_per_sm > 32) return CSD_ERR_INVALID_ARG;
    if (block_threads != 0 && (block_threads < 32 || block_threads > 1024 || block_threads % 32 != 0)) return CSD_ERR_INVALID_ARG;
    chain_break();
    g_chunk_bytes_override = chunk_bytes;
    g_ctas_per_sm_override = ctas_per_sm;
    g_block_threads_override = block_threads;
    return CSD_OK;
}

csd_status_t csd_set_overlap(int enable)
{
    chain_break();
    g_overlap_steps = enable ? 1 : 0;
    return CSD_OK;
}

const char *csd_status_string(csd_status_t status)
{
    switch (status) {
        case CSD_OK: return "ok";
        case CSD_ERR_INVALID_ARG: return "invalid argument";
        case CSD_ERR_CUDA: return "CUDA error";
        case CSD_ERR_OOM: return "out of memory";
        case CSD_ERR_UNSUPPORTED: return "unsupported shape";
        case CSD_ERR_WORKSPACE: return "workspace too small or misaligned";
        case CSD_ERR_IO: return "file cannot be opened, read or written, or is not a memory file";
    }
    return "unknown status";
}

}  // extern "C"
