// C ABI of the CFGzip decode-step library: argument checks, partition tables, launch
// planning. The declarations and their contracts are in include/cfgzip.h.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "cfgzip.h"
#include "cfgzip_kernels.cuh"

using namespace cfgzip;

namespace {

struct Part {
    bool live = false;
    int32_t V = 0, K = 0, KW = 0, VW = 0;
    void* block = nullptr;  // one device allocation holding every table of the partition
    PartDev dev{};
    std::vector<int32_t> sizes;  // host copy of the class sizes (cfgzip_choose_mode)
};

constexpr size_t kPartialSlots = size_t(1) << 18;  // 4 MB of (max, sum, pos) slots
constexpr size_t kFiltSmem = size_t(kFiltList) * 16;  // candidate list of the filtered sampling kernel
constexpr int kTwoOctetItemsPerWarp = 3;           // bf16: two octets per lane from this many work items per warp on
constexpr int kDefaultRows = 16384;

}  // namespace

// Scratch of cfgzip_step_noalloc: lives in the library image, one copy on every GPU that loads it.
constexpr int kNoAllocMaxRows = 1024;
constexpr int kNoAllocMaxSplits = 64;
struct NoAllocScratch {
    Partial partials[kNoAllocMaxRows * kNoAllocMaxSplits];  // 1 MiB
    unsigned int tickets[kNoAllocMaxRows];                  // 4 KiB
};
static __device__ __align__(256) NoAllocScratch g_noalloc_scratch;

struct cfgzip_ctx {
    int device = 0;
    int sm_count = 0;
    int smem_optin = 0;
    std::vector<Part> parts;
    PartDev* d_parts = nullptr;
    Partial* d_partials = nullptr;
    unsigned int* d_tickets = nullptr;  // reserved_rows entries
    int32_t* d_status = nullptr;        // 3 counters
    int32_t* d_group_part = nullptr;
    int32_t* d_group_rows = nullptr;
    int32_t* d_n_groups = nullptr;
    int32_t* d_row_mode = nullptr;      // automatic mode: which rows the class-list kernel has finished
    int32_t reserved_rows = 0;
    int32_t max_groups = 0;
    // staging for cfgzip_decode_step_host
    void* st_logits = nullptr;
    size_t st_logits_bytes = 0;
    uint32_t* st_cm = nullptr;
    size_t st_cm_bytes = 0;
    uint32_t* st_vm = nullptr;
    size_t st_vm_bytes = 0;
    int32_t* st_small = nullptr;  // row_part, argmax, rep, lse, logp_argmax: 5 arrays of st_rows
    int32_t st_rows = 0;
    int32_t* st_small_host = nullptr;  // pinned mirror of the four result arrays: they come back in one copy
    int64_t launches = 0;
    // row plan kept by cfgzip_plan_rows (valid until anything overwrites the plan buffers or the partitions change)
    bool plan_valid = false;
    bool plan_in_use = false;  // set for the duration of a call that passed CFGZIP_ROWS_AS_PLANNED
    const int32_t* plan_row_part = nullptr;
    int32_t plan_B = 0, plan_V = 0;
    // tuning
    int32_t ctas_per_sm = 4;
    int32_t token_warps = 0;
    int32_t row_warps = 0;
    int32_t pdl = 1;
    bool pdl_now = true;      // set per call: programmatic dependent launch only pays for short kernels
    int cluster_now = 1;      // set around a launch: blocks per thread-block cluster
    int prefetch_items = 4;   // work items per warp of the pipelined kernel asked into the L2 before its wait
    int prefetch_min_mbytes = 48;  // ... for steps of at least this many megabytes of logits
    bool prefetch_now = false;     // set per call beside pdl_now
    int rotate = 1;           // the chunk deal of the pipelined kernel starts at another warp slot for every row batch
    // cuTensorMapEncodeTiled, looked up through the runtime (no link against the driver library)
    CUresult (*encode_tiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill) = nullptr;
    int32_t pipeline = 1;     // bulk-copy pipelined dense kernel for aligned logits
    int32_t tensor_map = 1;   // tiled 2-D copies for row batches that are consecutive rows
    int32_t pipe_warps = 16;
    int32_t pipe_depth = 2;
    bool pipe_depth_set = false;  // the knob was set: no automatic third stage
    int32_t waves = 1;        // pipelined kernel: blocks launched per resident block slot
    int32_t spread = 1;       // pad the shared memory of one-block-per-SM launches so that blocks cannot share an SM
    int32_t stage_alias = 0;  // 1: always lay the class-mask staging area over the rings (default: only where it buys warps)
    int32_t lane_octets = 0;  // bf16 pipelined kernel: octets per lane and row (0 = automatic, 1, 2)
    int32_t auto_permille = -1;  // automatic mode: groups that allow under this many thousandths of their tokens go to the
                                 // class lists; -1 = by element type (measured break-even: f32 40, bf16 10)
    int64_t auto_min_bytes = -1;  // automatic mode on device-resident masks: steps of at least this many bytes of logits let the
                                  // GPU choose (one more launch); -1 = never (dense): the choice from host masks costs nothing
    int32_t fold = 0;         // pipelined kernel: the last block of a row group writes the rows' results (one launch per step)
    int32_t expire_test = 0;  // test hook: the pipelined kernel reports its first completed wait as run out
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

inline int ceil_div(int64_t a, int64_t b) { return int((a + b - 1) / b); }

template <typename... KArgs, typename... Args>
int launch(cfgzip_ctx* ctx, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
           Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (ctx->pdl == 2 || (ctx->pdl && ctx->pdl_now)) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    if (ctx->cluster_now > 1) {  // neighbouring blocks along x form a thread-block cluster
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = unsigned(ctx->cluster_now);
        attr[n_attr].val.clusterDim.y = 1;
        attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = unsigned(n_attr);
    if (cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...) != cudaSuccess) {
        cudaGetLastError();
        return CFGZIP_E_CUDA;
    }
    ctx->launches += 1;
    return CFGZIP_OK;
}

template <typename K>
int ensure_smem(K kernel, size_t bytes) {
    if (bytes <= 48 * 1024) return CFGZIP_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bytes)) != cudaSuccess) {
        cudaGetLastError();
        return CFGZIP_E_CUDA;
    }
    return CFGZIP_OK;
}

int check_partition_host(const int32_t* c, int32_t V, const int32_t* r, int32_t K) {
    if (!c || !r || V <= 0 || K <= 0 || K > V) return CFGZIP_E_ARG;
    std::vector<uint8_t> seen(size_t(K), 0);
    for (int32_t i = 0; i < V; ++i) {
        if (c[i] < 0 || c[i] >= K) return CFGZIP_E_PARTITION;
        seen[size_t(c[i])] = 1;
    }
    for (int32_t k = 0; k < K; ++k) {
        if (!seen[size_t(k)]) return CFGZIP_E_PARTITION;
        if (r[k] < 0 || r[k] >= V || c[r[k]] != k) return CFGZIP_E_PARTITION;
    }
    return CFGZIP_OK;
}

void build_class_lists_host(const int32_t* c, int32_t V, int32_t K, int32_t* off, int32_t* tok) {
    std::fill(off, off + K + 1, 0);
    for (int32_t i = 0; i < V; ++i) off[c[i] + 1] += 1;
    for (int32_t k = 0; k < K; ++k) off[k + 1] += off[k];
    std::vector<int32_t> cursor(off, off + K);
    for (int32_t i = 0; i < V; ++i) tok[cursor[size_t(c[i])]++] = i;  // ascending ids inside a class
}

// Everything a per-step call needs to know about the partitions it may touch.
struct PartSet {
    int32_t V = 0, VW = 0, maxK = 0, maxKW = 0, n_live_same_v = 0;
    bool all_c16 = true;
    bool all_kw_mult4 = true;
};

int resolve_parts(cfgzip_ctx* ctx, cfgzip_part_id part0, bool mixed, PartSet* ps) {
    if (part0 < 0 || size_t(part0) >= ctx->parts.size() || !ctx->parts[size_t(part0)].live) return CFGZIP_E_RANGE;
    const Part& p0 = ctx->parts[size_t(part0)];
    ps->V = p0.V;
    ps->VW = p0.VW;
    if (!mixed) {
        ps->maxK = p0.K;
        ps->maxKW = p0.KW;
        ps->n_live_same_v = 1;
        ps->all_c16 = p0.dev.c16 != nullptr;
        ps->all_kw_mult4 = (p0.KW % 4) == 0;
        return CFGZIP_OK;
    }
    for (const Part& p : ctx->parts) {
        if (!p.live || p.V != p0.V) continue;
        ps->maxK = std::max(ps->maxK, p.K);
        ps->maxKW = std::max(ps->maxKW, p.KW);
        ps->n_live_same_v += 1;
        ps->all_c16 = ps->all_c16 && p.dev.c16 != nullptr;
        ps->all_kw_mult4 = ps->all_kw_mult4 && (p.KW % 4) == 0;
    }
    return CFGZIP_OK;
}

bool aligned32(const void* p, int64_t row_stride_elems, int elem_size) {
    return (reinterpret_cast<uintptr_t>(p) & 31u) == 0 && ((row_stride_elems * elem_size) & 31) == 0;
}

bool aligned16(const void* p, int64_t row_stride_elems, int elem_size) {
    return (reinterpret_cast<uintptr_t>(p) & 15u) == 0 && ((row_stride_elems * elem_size) & 15) == 0;
}

size_t dense_smem_bytes(int table_words, int n_warps, int stage_stride) {
    (void)n_warps;
    return size_t(table_words) * 4 + kGroupRows * 4 + size_t(stage_stride) * kGroupRows * 4;
}

// Launch shape of the dense kernels.
struct DensePlan {
    int S = 1, per_split = 0, WT = 4, threads = 128, table_words = 0, stage_stride = 0;
    int depth = 0;       // > 0: pipelined kernel with this many stages per warp
    int cm_bulk = 0;     // pipelined kernel: class masks staged by bulk copies
    int stage_alias = 0; // pipelined kernel: staging area over the start of the rings
    int hold_warps = 0;
    int ctas_per_sm = 1; // blocks per SM the launch was sized for
    int opl = 1;         // pipelined kernel: octets per lane and row (2: bf16 chunks of 512 tokens)
    int fold = 0;        // pipelined kernel: results written by the last block of each group (no finalize launch)
    int fold_off = 0;    // fold: offset of the block's shared (row, warp) states, 0 = warps publish to the scratch directly
    int slots = 0;       // states per row in the global scratch
    size_t smem = 0;
    int n_groups_ub = 1;
    bool use_plan_kernel = false;
    bool ok = false;  // false: the dense kernels cannot run this call (generic path instead)
};

// alias: the class-mask staging area shares the space of the rings (it is dead once the table is built)
size_t pipe_smem_bytes(int table_words, int n_warps, int depth, int stage_bytes, int stage_stride, bool alias = false) {
    const size_t rings = size_t(n_warps) * depth * stage_bytes, staging = size_t(stage_stride) * kGroupRows * 4;
    return size_t(table_words) * 4 + kGroupRows * 4 + ((size_t(n_warps) * depth * 12 + 127) & ~size_t(127)) +
           (alias ? std::max(rings, staging) : rings + staging);
}

// Launch shape of the register-based dense kernels.
// units: octets (fused) or 32-token words (expand); unit_chunk: units one warp covers per iteration.
DensePlan plan_dense(cfgzip_ctx* ctx, const PartSet& ps, int32_t B, bool mixed, int units, int unit_chunk,
                     bool fused) {
    DensePlan d;
    d.table_words = (ps.maxKW + 1) * 32;
    d.use_plan_kernel = mixed;
    d.n_groups_ub = mixed ? ceil_div(B, kGroupRows) + ps.n_live_same_v : ceil_div(B, kGroupRows);
    if (!ps.all_c16) return d;
    if (dense_smem_bytes(d.table_words, 8, 0) > size_t(ctx->smem_optin) - 2048) return d;
    if (mixed && (B > ctx->reserved_rows || d.n_groups_ub > ctx->max_groups)) return d;
    const int ctas_per_sm = ctx->ctas_per_sm;
    // stage the class masks through shared memory while that keeps a block under 64 KB
    if (dense_smem_bytes(d.table_words, 8, ps.maxKW | 1) <= 64 * 1024) d.stage_stride = ps.maxKW | 1;
    d.ctas_per_sm = ctas_per_sm;
    const int target = ctx->sm_count * ctas_per_sm;
    const int n_chunks = ceil_div(units, unit_chunk);
    const int s0 = std::max(1, target / d.n_groups_ub);
    int cps = ceil_div(n_chunks, s0);  // chunks per block
    int WR = 1;
    if (fused) {
        WR = ctx->row_warps ? ctx->row_warps : (cps <= 2 ? 4 : 1);
        if (WR != 1 && WR != 2 && WR != 4) WR = 1;
        d.WT = ctx->token_warps ? ctx->token_warps : (WR == 4 ? std::min(cps, 2) : (WR == 2 ? 2 : 4));
        d.WT = std::max(1, std::min(d.WT, 8 / WR));
        d.threads = d.WT * WR * 32;
    } else {
        d.WT = 8;
        d.threads = 256;
    }
    for (;;) {
        d.S = ceil_div(n_chunks, cps);
        if (!fused || size_t(d.n_groups_ub) * kGroupRows * (size_t(d.S) * d.WT + 1) <= kPartialSlots) break;
        if (cps >= n_chunks) return d;
        cps *= 2;
    }
    d.per_split = cps * unit_chunk;
    d.slots = d.S * d.WT + 1;
    d.smem = dense_smem_bytes(d.table_words, fused ? d.threads / 32 : 0, d.stage_stride);
    d.ok = true;
    return d;
}

// Launch shape of the pipelined fused kernel. A block takes per_split octets (any number, not only
// whole 32-octet chunks) of one row group, so that the blocks of a step fill the SMs evenly.
DensePlan plan_pipe_opl(cfgzip_ctx* ctx, const PartSet& ps, int32_t B, bool mixed, int elem_size, bool cm_bulk_ok, int opl) {
    DensePlan d;
    d.opl = opl;
    d.table_words = (ps.maxKW + 1) * 32;
    d.use_plan_kernel = mixed;
    d.n_groups_ub = mixed ? ceil_div(B, kGroupRows) + ps.n_live_same_v : ceil_div(B, kGroupRows);
    if (!ps.all_c16 || !ctx->pipeline) return d;
    if (mixed && (B > ctx->reserved_rows || d.n_groups_ub > ctx->max_groups)) return d;
    const int chunk_octets = 32 * opl;
    const int stage_bytes = 8 * chunk_octets * 8 * elem_size + chunk_octets * 16;
    const size_t cap = size_t(ctx->smem_optin) - 2048;  // room for the kernel's static shared memory
    // two octets per lane: the variant is compiled for at most 12 warps (its stages are twice as large and it needs
    // more registers per thread)
    int n_warps = opl == 2 ? std::min(ctx->pipe_warps, 12) : ctx->pipe_warps, depth = ctx->pipe_depth;
    const int max_warps = n_warps;
    d.cm_bulk = cm_bulk_ok && ps.all_kw_mult4;
    int stride = d.cm_bulk ? ps.maxKW + (ps.maxKW % 8 == 0 ? 4 : 8) : (ps.maxKW | 1);
    auto fits = [&](int warps, int stages, bool over_rings) {
        return pipe_smem_bytes(d.table_words, warps, stages, stage_bytes, stride, over_rings) <= cap;
    };
    bool alias = ctx->stage_alias != 0;
    bool settled = false;
    // Long steps (twenty or more work items per warp) gain from a third stage where sharing the staging area makes
    // room for it (measured at V = 128256, bf16: B = 1024 -0.7 %, B = 2048 -1.4 %; B = 256 .. 512 lose 1 to 2 % to
    // the late start of the first warps).
    if (!ctx->pipe_depth_set && depth < 3 && fits(n_warps, 3, true)) {
        const int64_t blocks = int64_t(ctx->sm_count) * ctx->waves;
        const int64_t items = int64_t(ceil_div(B, kGroupRows)) * ceil_div(ps.V >> 3, chunk_octets) *
                              ceil_div(std::min<int>(B, kGroupRows), kBatchRows);
        if (items >= 20 * blocks * n_warps) {
            depth = 3;
            alias = true;
            settled = true;
        }
    }
    // Otherwise: the most warps (down to 8: a staged class-mask fetch is worth giving up warps for when the class
    // table is large) for which the staging area of the class masks fits, beside the rings of all warps or, where
    // it does not, laid over the first rings (their warps then start copying after the table is built).
    if (!settled) {
        const int step_down = opl == 2 ? 1 : 4;
        int w = n_warps;
        for (; w >= std::min(8, max_warps); w -= step_down) {
            if (ctx->stage_alias == 0 && fits(w, 2, false)) { alias = false; break; }
            if (fits(w, 2, true)) { alias = true; break; }
        }
        if (w >= std::min(8, max_warps)) {
            n_warps = w;
        } else {  // no staging: every lane reads its row's class-mask words from global memory
            n_warps = max_warps;
            stride = 0;
            d.cm_bulk = 0;
            alias = false;
        }
    }
    while (depth > 2 && pipe_smem_bytes(d.table_words, n_warps, depth, stage_bytes, stride, alias) > cap) --depth;
    while (n_warps > 4 && pipe_smem_bytes(d.table_words, n_warps, depth, stage_bytes, stride, alias) > cap)
        n_warps -= opl == 2 ? 1 : 2;
    size_t smem = pipe_smem_bytes(d.table_words, n_warps, depth, stage_bytes, stride, alias);
    if (smem > cap) return d;
    if (stride == 0) alias = false;
    d.depth = depth;
    d.stage_stride = stride;
    const int fit = std::max(1, int((cap + 1024) / (smem + 1024)));
    d.ctas_per_sm = opl == 2 ? 1 : std::min(ctx->ctas_per_sm, fit);
    const int target = ctx->sm_count * d.ctas_per_sm * ctx->waves;
    const int n_oct = 4 * ps.VW;
    // blocks of groups that turn out not to exist leave at once, so size the split for the fewest
    // groups the batch can have
    const int s0 = std::max(1, target / ceil_div(B, kGroupRows));
    int per = std::max(chunk_octets, ceil_div(n_oct, s0));
    // Warps go side by side along the vocabulary first (long contiguous runs per row are kind to
    // DRAM); only when a block has fewer chunks than warps do warps split the row batches.
    const int chunks = ceil_div(per, chunk_octets);
    int WR = ctx->row_warps;
    if (!WR) {
        WR = 1;
        while (WR < 4 && chunks * WR * 2 <= n_warps) WR <<= 1;
    }
    while (WR > 1 && (WR - 1) * kBatchRows >= std::min<int>(B, kGroupRows)) WR >>= 1;
    if ((WR != 1 && WR != 2 && WR != 4)) WR = 1;
    d.WT = ctx->token_warps ? ctx->token_warps : n_warps / WR;
    d.WT = std::max(1, std::min(std::min(d.WT, max_warps / WR), chunks));
    d.threads = d.WT * WR * 32;
    for (;;) {
        d.S = ceil_div(n_oct, per);
        if (size_t(d.n_groups_ub) * kGroupRows * (size_t(d.S) * d.WT + 1) <= kPartialSlots) break;
        if (per >= n_oct) return d;
        per *= 2;
    }
    d.per_split = per;
    d.stage_alias = alias ? 1 : 0;
    d.hold_warps = alias ? std::min(d.threads / 32, ceil_div(int64_t(d.stage_stride) * kGroupRows * 4, int64_t(d.depth) * stage_bytes)) : 0;
    d.smem = pipe_smem_bytes(d.table_words, d.threads / 32, d.depth, stage_bytes, d.stage_stride, alias);
    d.slots = d.S * d.WT + 1;
    // One launch per step: the last block of a group folds the group's states. Where shared memory has room the
    // warps of a block first merge their states there (one state per row and block reaches the scratch); otherwise
    // the warps publish directly, which is only taken while a row has few states.
    if (ctx->fold) {  // 1: fold in the kernel; 2: only merge the states of a block's warps before they are published
        const size_t block_states = size_t(kGroupRows) * (d.WT + 1) * sizeof(Partial);
        if (d.smem + block_states <= cap) {
            d.fold = ctx->fold == 1;
            d.fold_off = int(d.smem);
            d.smem += block_states;
            d.slots = d.S;
        } else if (d.slots <= 256) {
            d.fold = ctx->fold == 1;
        }
    }
    // A launch sized for one block per SM asks for more than half of an SM's shared memory even when its few warps
    // need less, so that two of its blocks never share an SM while another SM stays empty (measured at B = 8 .. 24:
    // 10.2 -> 7.7 us, 10.1 -> 8.8 us, 12.4 -> 10.6 us).
    if (d.ctas_per_sm == 1 && ctx->spread) d.smem = std::max(d.smem, cap / 2 + 1024);
    d.ok = true;
    return d;
}

// Launch shape of the pipelined fused kernel. bf16 rows may be streamed with one octet (16 bytes) or two octets
// (32 bytes) per lane and row; two octets halve the per-row bookkeeping but double a work item, so they are taken
// only when every warp of the launch still gets several items.
DensePlan plan_pipe(cfgzip_ctx* ctx, const PartSet& ps, int32_t B, bool mixed, int elem_size, bool cm_bulk_ok) {
    const DensePlan one = plan_pipe_opl(ctx, ps, B, mixed, elem_size, cm_bulk_ok, 1);
    if (elem_size != 2 || ctx->lane_octets == 1) return one;
    const DensePlan two = plan_pipe_opl(ctx, ps, B, mixed, elem_size, cm_bulk_ok, 2);
    if (!two.ok) return one;
    if (!one.ok || ctx->lane_octets == 2) return two;
    if (ctx->lane_octets == 0) return one;
    const int64_t items = int64_t(ceil_div(B, kGroupRows)) * ceil_div(ps.V >> 3, 64) *
                          ceil_div(std::min<int>(B, kGroupRows), kBatchRows);
    const int64_t warps = int64_t(ctx->sm_count) * ctx->waves * (two.threads / 32);
    return items >= kTwoOctetItemsPerWarp * warps ? two : one;
}

// A call may pass CFGZIP_ROWS_AS_PLANNED for its row -> partition vector: it then means the vector given to the
// last cfgzip_plan_rows, whose grouping is still in the plan buffers.
int resolve_row_part(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t** row_part, int32_t B, bool* planned) {
    *planned = false;
    if (*row_part != CFGZIP_ROWS_AS_PLANNED) return CFGZIP_OK;
    if (!ctx) return CFGZIP_E_ARG;
    if (!ctx->plan_valid || ctx->plan_B != B || part0 < 0 || size_t(part0) >= ctx->parts.size() ||
        !ctx->parts[size_t(part0)].live || ctx->parts[size_t(part0)].V != ctx->plan_V)
        return CFGZIP_E_ARG;
    *row_part = ctx->plan_row_part;
    *planned = true;
    return CFGZIP_OK;
}

struct PlanUse {  // marks the kept plan as in use for the lifetime of a call
    cfgzip_ctx* ctx;
    PlanUse(cfgzip_ctx* c, bool planned) : ctx(c) { if (ctx) ctx->plan_in_use = planned; }
    ~PlanUse() { if (ctx) ctx->plan_in_use = false; }
};

int check_step_args(cfgzip_ctx* ctx, const uint32_t* class_mask, int64_t cm_stride, int32_t B, int mode) {
    if (!ctx || B < 0) return CFGZIP_E_ARG;
    if (mode != CFGZIP_AUTO && mode != CFGZIP_DENSE && mode != CFGZIP_SPARSE) return CFGZIP_E_ARG;
    if (B > 0 && (!class_mask || cm_stride <= 0)) return CFGZIP_E_ARG;
    return CFGZIP_OK;
}

int run_plan_kernel(cfgzip_ctx* ctx, const int32_t* row_part, int32_t B, int32_t V, const DensePlan& d,
                    cudaStream_t st) {
    if (ctx->plan_in_use) return CFGZIP_OK;  // the call runs on the grouping cfgzip_plan_rows left in the buffers
    ctx->plan_valid = false;                 // this launch overwrites them
    return launch(ctx, k_plan_rows, dim3(1), dim3(1024), 0, st, (const PartDev*)ctx->d_parts, int(ctx->parts.size()),
                  row_part, int(B), int(V), d.n_groups_ub, ctx->d_group_part, ctx->d_group_rows, ctx->d_n_groups,
                  ctx->d_status);
}

void fill_groups(cfgzip_ctx* ctx, StepArgs& a, const DensePlan& d) {
    if (d.use_plan_kernel) {
        a.group_part = ctx->d_group_part;
        a.group_rows = ctx->d_group_rows;
        a.n_groups = ctx->d_n_groups;
    } else {
        a.group_part = nullptr;
        a.group_rows = nullptr;
        a.n_groups = nullptr;
    }
    a.S = d.S;
    a.per_split = d.per_split;
    a.WT = d.WT;
    a.table_words = d.table_words;
    a.stage_stride = d.stage_stride;
    a.depth = d.depth;
    a.cm_bulk = d.cm_bulk;
    a.stage_alias = d.stage_alias;
    a.hold_warps = d.hold_warps;
    a.slots = d.slots;
    a.fold = d.fold;
    a.fold_off = d.fold_off;
    a.chunk_tokens = 256 * d.opl;
    // Only a programmatic launch runs ahead of the kernel in front, and only from about 48 MB of logits on does asking
    // ahead pay (measured: B = 256 -3.6 %, qwen-size -2.3 %, B = 512 -1.6 %; shorter steps lose, B = 32 +7 %: the
    // requests compete with the loads of the kernel in front, whose end the step waits for).
    a.prefetch_items = ((ctx->pdl == 2 || (ctx->pdl && ctx->pdl_now)) && ctx->prefetch_now) ? ctx->prefetch_items : 0;
    a.rot_chunks = ctx->rotate ? std::max(1, d.S * d.WT / ceil_div(std::min<int>(a.B, kGroupRows), kBatchRows)) : 0;
    a.expire_test = ctx->expire_test;
    a.p0 = ctx->parts[size_t(a.part0)].dev;
}

// Sparse launch shape: S blocks per row, each owning per_split vocab-mask words in shared memory.
bool plan_sparse(cfgzip_ctx* ctx, const PartSet& ps, int32_t B, bool fused, int* S, int* per_split) {
    const int target = ctx->sm_count * ctx->ctas_per_sm;
    int s = std::max(1, target / std::max(B, 1));
    s = std::min(s, std::max(1, ps.VW / 256));
    const int max_words = (ctx->smem_optin - 8192) / 4;
    for (;;) {
        *per_split = ((ceil_div(ps.VW, s) + 3) / 4) * 4;
        if (*per_split <= max_words) break;
        s *= 2;
    }
    *S = ceil_div(ps.VW, *per_split);
    if (fused && *S > 1) {
        if (B > ctx->reserved_rows) return false;
        if (size_t(B) * size_t(*S) > kPartialSlots) {
            // fall back to one block per row if shared memory allows it
            *per_split = ((ps.VW + 3) / 4) * 4;
            *S = 1;
            if (*per_split > max_words) return false;
        }
    }
    return true;
}

// Shared memory a per-row kernel (one small block per row) asks for without using it: when its blocks are no more
// than the SMs, more than half of an SM's shared memory keeps every block on an SM of its own. Measured on the
// finalize kernel: B = 32 step 12.0 -> 11.4 us, B = 64 16.3 -> 15.4, B = 128 22.1 -> 21.2; nothing from 256 rows on,
// and a loss under 32 rows, where most of the 32 blocks leave at once.
size_t row_blocks_pad(const cfgzip_ctx* ctx, unsigned rows_grid, int32_t B) {
    if (!ctx->spread || B < kGroupRows || rows_grid > unsigned(ctx->sm_count)) return 0;
    return size_t(ctx->smem_optin) / 2 + 1024;
}

// The pipelined streaming kernel for a planned step (d.depth > 0; `a` filled by fill_groups).
template <int DT>
int launch_pipe(cfgzip_ctx* ctx, const StepArgs& a, const DensePlan& d, dim3 grid, dim3 block, cudaStream_t st) {
    int rc;
    // rows of a batch are consecutive unless the plan kernel regrouped them: then one tiled
    // 2-D copy (box 256 elements x 8 rows) brings a whole batch
    CUtensorMap tmap;
    std::memset(&tmap, 0, sizeof tmap);
    bool tiled = false;
    if (!d.use_plan_kernel && ctx->tensor_map && ctx->encode_tiled && a.V >= 256 &&
        a.row_stride * (DT == kBF16 ? 2 : 4) < (int64_t(1) << 32) && a.vm_stride * 4 < (int64_t(1) << 32)) {
        const cuuint64_t dims[2] = {cuuint64_t(a.V), cuuint64_t(a.B)};
        const cuuint64_t strides[1] = {cuuint64_t(a.row_stride) * (DT == kBF16 ? 2 : 4)};
        const cuuint32_t box[2] = {256, 8};
        const cuuint32_t estr[2] = {1, 1};
        tiled = ctx->encode_tiled(&tmap, DT == kBF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                  2, a.logits, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    }
    void (*kern)(StepArgs, CUtensorMap);
    const bool tempered = a.u != nullptr;  // only a sampling step has a temperature
    constexpr int kTwo = DT == kBF16 ? 2 : 1;  // f32 lanes always take one octet (32 bytes)
#define CFGZIP_PIPE_VARIANT(OPL, LBT, MINB)                                                                         \
    (tempered ? (tiled ? k_step_dense_pipe<DT, OPL, true, LBT, MINB, true> : k_step_dense_pipe<DT, OPL, false, LBT, MINB, true>) \
              : (tiled ? k_step_dense_pipe<DT, OPL, true, LBT, MINB, false> : k_step_dense_pipe<DT, OPL, false, LBT, MINB, false>))
    if (d.opl == 2 && kTwo == 2 && d.threads <= 384)
        kern = CFGZIP_PIPE_VARIANT(kTwo, 384, 1);
    else if (d.opl != 1)
        return CFGZIP_E_ARG;  // the planner never asks for this
    else if (d.threads <= 256 && d.ctas_per_sm >= 3)
        kern = CFGZIP_PIPE_VARIANT(1, 256, 3);
    else if (d.threads <= 320 && d.ctas_per_sm >= 2)
        kern = CFGZIP_PIPE_VARIANT(1, 320, 2);
    else
        kern = CFGZIP_PIPE_VARIANT(1, 512, 1);
#undef CFGZIP_PIPE_VARIANT
    if ((rc = ensure_smem(kern, d.smem)) != CFGZIP_OK) return rc;
    return launch(ctx, kern, grid, block, d.smem, st, a, tmap);
}

template <int DT>
int launch_fused(cfgzip_ctx* ctx, StepArgs& a, const PartSet& ps, bool mixed, int mode, bool aligned, float* logp_full,
                 cudaStream_t st) {
    int rc;
    if (!aligned) {
        // rows off the 16-byte grid: the per-row kernel with element-wise accesses
        rc = launch(ctx, k_step_generic<DT, true>, dim3(unsigned(a.B)), dim3(256), 0, st, a);
    } else if (mode == CFGZIP_SPARSE) {
        int S, per_split;
        if (plan_sparse(ctx, ps, a.B, true, &S, &per_split)) {
            a.S = S;
            a.per_split = per_split;
            const size_t smem = size_t(per_split) * 4;
            auto kern = k_step_sparse<DT, true>;
            if ((rc = ensure_smem(kern, smem)) != CFGZIP_OK) return rc;
            rc = launch(ctx, kern, dim3(unsigned(a.B) * unsigned(S)), dim3(256), smem, st, a);
        } else {
            rc = launch(ctx, k_step_generic<DT, true>, dim3(unsigned(a.B)), dim3(256), 0, st, a);
        }
    } else {
        const bool cm_bulk_ok = (reinterpret_cast<uintptr_t>(a.class_mask) & 15u) == 0 && (a.cm_stride & 3) == 0;
        DensePlan d = plan_pipe(ctx, ps, a.B, mixed, DT == kBF16 ? 2 : 4, cm_bulk_ok);
        if (!d.ok) d = plan_dense(ctx, ps, a.B, mixed, 4 * ps.VW, 32, true);
        if (d.ok) {
            if (d.use_plan_kernel && (rc = run_plan_kernel(ctx, a.row_part, a.B, a.V, d, st)) != CFGZIP_OK) return rc;
            // Automatic mode on a long step: the class-list kernel runs first, keeps the row batches (the 8 rows the
            // gather kernel streams together) that allow few tokens (it never reads a logit that is not allowed) and
            // marks the others for the gather kernel behind it.
            // Short steps are dense outright (the extra launch would cost more than the class lists can save).
            int sp_S = 0, sp_per = 0;
            const int permille = ctx->auto_permille >= 0 ? ctx->auto_permille : (DT == kBF16 ? 10 : 40);
            const bool choose = mode == CFGZIP_AUTO && d.depth > 0 && permille > 0 && ctx->d_row_mode != nullptr &&
                                a.B <= ctx->reserved_rows && ctx->auto_min_bytes >= 0 &&
                                int64_t(a.B) * a.V * (DT == kBF16 ? 2 : 4) >= ctx->auto_min_bytes &&
                                plan_sparse(ctx, ps, a.B, true, &sp_S, &sp_per);
            if (choose) {
                if (d.fold_off) d.smem -= size_t(kGroupRows) * (d.WT + 1) * sizeof(Partial);
                d.fold = d.fold_off = 0;                // the tickets belong to the class-list kernel here
                d.slots = d.S * d.WT + 1;
            }
            fill_groups(ctx, a, d);
            if (choose) {
                a.row_mode = ctx->d_row_mode;
                a.auto_permille = permille;
                StepArgs b = a;  // one row per S blocks
                b.S = sp_S;
                b.per_split = sp_per;
                const size_t smem = size_t(sp_per) * 4;
                auto kern = k_step_sparse<DT, true>;
                if ((rc = ensure_smem(kern, smem)) != CFGZIP_OK) return rc;
                if ((rc = launch(ctx, kern, dim3(unsigned(d.n_groups_ub) * kGroupRows * unsigned(sp_S)), dim3(256), smem, st, b)) !=
                    CFGZIP_OK)
                    return rc;
            }
            const dim3 grid(unsigned(d.n_groups_ub) * unsigned(d.S)), block{unsigned(d.threads)};
            if (d.depth) {
                rc = launch_pipe<DT>(ctx, a, d, grid, block, st);
            } else {
                auto kern = k_step_dense<DT>;
                if ((rc = ensure_smem(kern, d.smem)) != CFGZIP_OK) return rc;
                rc = launch(ctx, kern, grid, block, d.smem, st, a);
            }
            // second kernel: one block per row folds the published states and writes the results (unless the
            // streaming kernel's last block of each group has done so)
            if (rc == CFGZIP_OK && !(d.depth && d.fold)) {
                if (a.slots <= kFinalizeWarpStates)  // few states per row: a warp per row
                    rc = launch(ctx, k_finalize_rows_warp<DT>, dim3(unsigned(d.n_groups_ub) * (kGroupRows / 8)), dim3(256), 0, st, a);
                else
                {
                    const unsigned rows_grid = unsigned(d.n_groups_ub) * kGroupRows;
                    const size_t pad = row_blocks_pad(ctx, rows_grid, a.B);
                    if (pad && (rc = ensure_smem(k_finalize_rows<DT>, pad)) != CFGZIP_OK) return rc;
                    rc = launch(ctx, k_finalize_rows<DT>, dim3(rows_grid), dim3(kFinalizeThreads), pad, st, a);
                }
            }
        } else {
            rc = launch(ctx, k_step_generic<DT, true>, dim3(unsigned(a.B)), dim3(256), 0, st, a);
        }
    }
    if (rc != CFGZIP_OK) return rc;
    if (logp_full) {
        const dim3 grid(unsigned(std::min(ceil_div(a.V, 256 * 4), 64)), unsigned(std::min<int32_t>(a.B, 65535)));
        rc = launch(ctx, k_logp_full<DT>, grid, dim3(256), 0, st, (const void*)a.logits, a.row_stride, int(a.B),
                    int(a.V), (const float*)a.lse, logp_full);
    }
    return rc;
}

// The draw of a sampling step with top-k / top-p. One block per row leaves most of the device idle on a short batch,
// so 4 or 2 blocks (a thread-block cluster) share a row while that many blocks still fit the device in one wave.
template <int DT>
int launch_filtered(cfgzip_ctx* ctx, const StepArgs& a, unsigned rows_grid, int aligned, int top_k, float top_p,
                    cudaStream_t st) {
    int rc;
    if ((rc = ensure_smem(k_sample_filtered<DT>, kFiltSmem)) != CFGZIP_OK) return rc;
    const unsigned sms = unsigned(std::max(ctx->sm_count, 1));
    const unsigned per_row = rows_grid * 4 <= sms ? 4u : (rows_grid * 2 <= sms ? 2u : 1u);
    ctx->cluster_now = int(per_row);
    rc = launch(ctx, k_sample_filtered<DT>, dim3(rows_grid * per_row), dim3(kFiltThreads), kFiltSmem, st, a, aligned, top_k,
                top_p);
    ctx->cluster_now = 1;
    if (rc != CFGZIP_OK && per_row > 1)  // a device that cannot place such a cluster: one block per row
        rc = launch(ctx, k_sample_filtered<DT>, dim3(rows_grid), dim3(kFiltThreads), kFiltSmem, st, a, aligned, top_k, top_p);
    return rc;
}

// A sampling step: the streaming kernel leaves the states of a row in token order, the sampling kernel
// (one block per row) draws the token. Rows off the 16-byte grid, and shapes the pipelined kernel does not
// take, go through the per-row kernel, whose single state per row stands for the whole row.
template <int DT>
int launch_sample(cfgzip_ctx* ctx, StepArgs& a, const PartSet& ps, bool mixed, bool aligned, int top_k, float top_p,
                  cudaStream_t st) {
    const bool filtered = top_k > 0 || top_p < 1.f;  // the draw is restricted to the most probable tokens
    int rc;
    DensePlan d;
    if (aligned) {
        const bool cm_bulk_ok = (reinterpret_cast<uintptr_t>(a.class_mask) & 15u) == 0 && (a.cm_stride & 3) == 0;
        d = plan_pipe(ctx, ps, a.B, mixed, DT == kBF16 ? 2 : 4, cm_bulk_ok);
    }
    if (d.ok && d.depth) {
        if (d.use_plan_kernel && (rc = run_plan_kernel(ctx, a.row_part, a.B, a.V, d, st)) != CFGZIP_OK) return rc;
        // a sampling step keeps one state per warp slot in token order and a kernel of its own for the draw
        if (d.fold_off) d.smem -= size_t(kGroupRows) * (d.WT + 1) * sizeof(Partial);
        d.fold = d.fold_off = 0;
        d.slots = d.S * d.WT + 1;
        fill_groups(ctx, a, d);
        const int n_chunks = ceil_div(ps.V >> 3, 32 * d.opl);
        a.run_chunks = std::max(1, ceil_div(n_chunks, d.S * d.WT));
        a.tail_state = 1;
        const dim3 grid(unsigned(d.n_groups_ub) * unsigned(d.S)), block{unsigned(d.threads)};
        if ((rc = launch_pipe<DT>(ctx, a, d, grid, block, st)) != CFGZIP_OK) return rc;
        const unsigned rows_grid = unsigned(d.n_groups_ub) * kGroupRows;
        if (filtered) return launch_filtered<DT>(ctx, a, rows_grid, 1, top_k, top_p, st);
        const size_t pad = row_blocks_pad(ctx, rows_grid, a.B);
        if (pad && (rc = ensure_smem(k_sample_rows<DT>, pad)) != CFGZIP_OK) return rc;
        return launch(ctx, k_sample_rows<DT>, dim3(rows_grid), dim3(kSampleThreads), pad, st, a, 1);
    }
    if (size_t(a.B) > kPartialSlots) return CFGZIP_E_NOMEM;
    a.group_part = nullptr;
    a.group_rows = nullptr;
    a.n_groups = nullptr;
    a.slots = 1;
    a.run_chunks = ceil_div(ps.V, 256);
    a.chunk_tokens = 256;
    a.tail_state = 0;
    a.p0 = ctx->parts[size_t(a.part0)].dev;
    if ((rc = launch(ctx, k_step_generic<DT, true>, dim3(unsigned(a.B)), dim3(256), 0, st, a)) != CFGZIP_OK) return rc;
    if (filtered)
        return launch_filtered<DT>(ctx, a, unsigned(ceil_div(a.B, kGroupRows)) * kGroupRows, aligned ? 1 : 0, top_k, top_p, st);
    return launch(ctx, k_sample_rows<DT>, dim3(unsigned(ceil_div(a.B, kGroupRows)) * kGroupRows), dim3(kSampleThreads), 0, st,
                  a, aligned ? 1 : 0);
}

int grow(void** p, size_t* have, size_t need) {
    if (need <= *have) return CFGZIP_OK;
    if (*p) cudaFree(*p);
    *p = nullptr;
    *have = 0;
    if (cudaMalloc(p, need) != cudaSuccess) {
        cudaGetLastError();
        return CFGZIP_E_NOMEM;
    }
    *have = need;
    return CFGZIP_OK;
}

}  // namespace

extern "C" {

const char* cfgzip_status_string(int status) {
    switch (status) {
        case CFGZIP_OK: return "CFGZIP_OK";
        case CFGZIP_E_ARG: return "CFGZIP_E_ARG: invalid argument";
        case CFGZIP_E_RANGE: return "CFGZIP_E_RANGE: id or size out of range";
        case CFGZIP_E_PARTITION: return "CFGZIP_E_PARTITION: c / r do not describe a partition";
        case CFGZIP_E_ALIGN: return "CFGZIP_E_ALIGN: misaligned buffer";
        case CFGZIP_E_CUDA: return "CFGZIP_E_CUDA: CUDA runtime error";
        case CFGZIP_E_NOMEM: return "CFGZIP_E_NOMEM: out of memory or capacity";
        default: return "CFGZIP: unknown status";
    }
}

int cfgzip_check_partition(const int32_t* token_to_class, int32_t V, const int32_t* class_to_rep, int32_t K) {
    return check_partition_host(token_to_class, V, class_to_rep, K);
}

int cfgzip_build_class_lists(const int32_t* token_to_class, int32_t V, int32_t K, int32_t* off, int32_t* tok) {
    if (!token_to_class || !off || !tok || V <= 0 || K <= 0 || K > V) return CFGZIP_E_ARG;
    for (int32_t i = 0; i < V; ++i)
        if (token_to_class[i] < 0 || token_to_class[i] >= K) return CFGZIP_E_PARTITION;
    build_class_lists_host(token_to_class, V, K, off, tok);
    return CFGZIP_OK;
}

int cfgzip_reserve_rows(cfgzip_ctx* ctx, int32_t max_rows) {
    if (!ctx || max_rows <= 0) return CFGZIP_E_ARG;
    if (max_rows <= ctx->reserved_rows) return CFGZIP_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    cudaDeviceSynchronize();
    ctx->plan_valid = false;
    cudaFree(ctx->d_tickets);
    cudaFree(ctx->d_group_part);
    cudaFree(ctx->d_group_rows);
    cudaFree(ctx->d_row_mode);
    ctx->d_tickets = nullptr;
    ctx->d_group_part = ctx->d_group_rows = ctx->d_row_mode = nullptr;
    ctx->reserved_rows = 0;
    const int32_t groups = ceil_div(max_rows, kGroupRows) + kMaxParts;
    const size_t tickets = size_t(std::max(max_rows, groups));
    if (cudaMalloc(&ctx->d_tickets, tickets * sizeof(unsigned int)) != cudaSuccess ||
        cudaMalloc(&ctx->d_group_part, size_t(groups) * sizeof(int32_t)) != cudaSuccess ||
        cudaMalloc(&ctx->d_group_rows, size_t(groups) * kGroupRows * sizeof(int32_t)) != cudaSuccess ||
        cudaMalloc(&ctx->d_row_mode, size_t(max_rows) * sizeof(int32_t)) != cudaSuccess) {
        cudaGetLastError();
        return CFGZIP_E_NOMEM;
    }
    cudaMemset(ctx->d_tickets, 0, tickets * sizeof(unsigned int));
    ctx->reserved_rows = max_rows;
    ctx->max_groups = groups;
    return CFGZIP_OK;
}

int cfgzip_create(int device, cfgzip_ctx** out) {
    if (!out) return CFGZIP_E_ARG;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) {
        cudaGetLastError();
        return CFGZIP_E_CUDA;
    }
    DeviceGuard guard(device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    cfgzip_ctx* ctx = new (std::nothrow) cfgzip_ctx();
    if (!ctx) return CFGZIP_E_NOMEM;
    ctx->device = device;
    cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
    cudaDeviceGetAttribute(&ctx->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            ctx->encode_tiled = reinterpret_cast<decltype(ctx->encode_tiled)>(fn);
        else
            cudaGetLastError();
    }
    bool ok = cudaMalloc(&ctx->d_parts, kMaxParts * sizeof(PartDev)) == cudaSuccess &&
              cudaMalloc(&ctx->d_partials, kPartialSlots * sizeof(Partial)) == cudaSuccess &&
              cudaMalloc(&ctx->d_status, 4 * sizeof(int32_t)) == cudaSuccess &&
              cudaMalloc(&ctx->d_n_groups, sizeof(int32_t)) == cudaSuccess;
    if (ok) {
        cudaMemset(ctx->d_parts, 0, kMaxParts * sizeof(PartDev));
        cudaMemset(ctx->d_status, 0, 4 * sizeof(int32_t));
        cudaMemset(ctx->d_n_groups, 0, sizeof(int32_t));
        ok = cfgzip_reserve_rows(ctx, kDefaultRows) == CFGZIP_OK;
    }
    if (!ok || cudaDeviceSynchronize() != cudaSuccess) {
        cudaGetLastError();
        cfgzip_destroy(ctx);
        return CFGZIP_E_NOMEM;
    }
    *out = ctx;
    return CFGZIP_OK;
}

int cfgzip_destroy(cfgzip_ctx* ctx) {
    if (!ctx) return CFGZIP_E_ARG;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    for (Part& p : ctx->parts)
        if (p.block) cudaFree(p.block);
    cudaFree(ctx->d_parts);
    cudaFree(ctx->d_partials);
    cudaFree(ctx->d_tickets);
    cudaFree(ctx->d_status);
    cudaFree(ctx->d_group_part);
    cudaFree(ctx->d_group_rows);
    cudaFree(ctx->d_row_mode);
    cudaFree(ctx->d_n_groups);
    cudaFree(ctx->st_logits);
    cudaFree(ctx->st_cm);
    cudaFree(ctx->st_vm);
    cudaFree(ctx->st_small);
    if (ctx->st_small_host) cudaFreeHost(ctx->st_small_host);
    cudaGetLastError();
    delete ctx;
    return CFGZIP_OK;
}

int cfgzip_load_partition(cfgzip_ctx* ctx, const int32_t* c, int32_t V, const int32_t* r, int32_t K, void* stream,
                          cfgzip_part_id* out_id) {
    if (!ctx || !out_id) return CFGZIP_E_ARG;
    int rc = check_partition_host(c, V, r, K);
    if (rc != CFGZIP_OK) return rc;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    size_t slot = 0;
    while (slot < ctx->parts.size() && ctx->parts[slot].live) ++slot;
    if (slot >= size_t(kMaxParts)) return CFGZIP_E_RANGE;
    const bool appended = slot == ctx->parts.size();
    if (appended) ctx->parts.emplace_back();

    Part p;
    p.V = V;
    p.K = K;
    p.KW = ceil_div(K, 32);
    p.VW = ceil_div(V, 32);
    const bool has16 = K <= 65535;  // the value K itself is the padding id
    // host image of the device block: c32 | r | off | tok | trep | c16 (16-byte aligned pieces)
    auto align4 = [](size_t n) { return (n + 3) & ~size_t(3); };
    const size_t n_c32 = align4(size_t(V)), n_r = align4(size_t(K)), n_off = align4(size_t(K) + 1), n_tok = align4(size_t(V));
    const size_t n_trep = align4(size_t(V));
    const size_t n_c16_words = has16 ? size_t(p.VW) * 16 : 0;  // 32*VW uint16 = 16*VW words
    std::vector<int32_t> img(n_c32 + n_r + n_off + n_tok + n_trep + n_c16_words, 0);
    int32_t* h_c32 = img.data();
    int32_t* h_r = h_c32 + n_c32;
    int32_t* h_off = h_r + n_r;
    int32_t* h_tok = h_off + n_off;
    int32_t* h_trep = h_tok + n_tok;
    uint16_t* h_c16 = reinterpret_cast<uint16_t*>(h_trep + n_trep);
    std::memcpy(h_c32, c, size_t(V) * 4);
    std::memcpy(h_r, r, size_t(K) * 4);
    build_class_lists_host(c, V, K, h_off, h_tok);
    p.sizes.resize(size_t(K));
    for (int32_t k = 0; k < K; ++k) p.sizes[size_t(k)] = h_off[k + 1] - h_off[k];
    for (int32_t i = 0; i < V; ++i) h_trep[i] = r[c[i]];
    if (has16) {
        for (int32_t i = 0; i < V; ++i) h_c16[i] = uint16_t(c[i]);
        for (int32_t i = V; i < 32 * p.VW; ++i) h_c16[i] = uint16_t(K);
    }
    if (cudaMalloc(&p.block, img.size() * 4) != cudaSuccess) {
        cudaGetLastError();
        if (appended) ctx->parts.pop_back();
        return CFGZIP_E_NOMEM;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t* d = static_cast<int32_t*>(p.block);
    p.dev.c32 = d;
    p.dev.r = d + n_c32;
    p.dev.off = d + n_c32 + n_r;
    p.dev.tok = d + n_c32 + n_r + n_off;
    p.dev.trep = d + n_c32 + n_r + n_off + n_tok;
    p.dev.c16 = has16 ? reinterpret_cast<const uint16_t*>(d + n_c32 + n_r + n_off + n_tok + n_trep) : nullptr;
    p.dev.K = K;
    p.dev.KW = p.KW;
    p.dev.V = V;
    p.dev.live = 1;
    p.live = true;
    bool ok = cudaMemcpyAsync(p.block, img.data(), img.size() * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaMemcpyAsync(ctx->d_parts + slot, &p.dev, sizeof(PartDev), cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaStreamSynchronize(st) == cudaSuccess;
    if (!ok) {
        // the descriptor may already be on the device: clear it before its tables are freed, so that no later
        // call finds a live slot that points at released memory
        cudaGetLastError();
        cudaStreamSynchronize(st);
        cudaMemset(ctx->d_parts + slot, 0, sizeof(PartDev));
        cudaDeviceSynchronize();
        cudaGetLastError();
        cudaFree(p.block);
        if (appended) ctx->parts.pop_back();
        return CFGZIP_E_CUDA;
    }
    ctx->parts[slot] = p;
    ctx->plan_valid = false;
    *out_id = cfgzip_part_id(slot);
    return CFGZIP_OK;
}

int cfgzip_free_partition(cfgzip_ctx* ctx, cfgzip_part_id id) {
    if (!ctx) return CFGZIP_E_ARG;
    if (id < 0 || size_t(id) >= ctx->parts.size() || !ctx->parts[size_t(id)].live) return CFGZIP_E_RANGE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    cudaDeviceSynchronize();
    ctx->plan_valid = false;
    Part& p = ctx->parts[size_t(id)];
    cudaFree(p.block);
    p = Part();
    cudaMemset(ctx->d_parts + id, 0, sizeof(PartDev));
    cudaDeviceSynchronize();
    return cudaGetLastError() == cudaSuccess ? CFGZIP_OK : CFGZIP_E_CUDA;
}

int cfgzip_expand_mask(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part, const uint32_t* class_mask,
                       int64_t class_stride_words, uint32_t* vocab_mask, int64_t vocab_stride_words, int32_t B,
                       int mode, void* stream) {
    int rc = check_step_args(ctx, class_mask, class_stride_words, B, mode);
    if (rc != CFGZIP_OK) return rc;
    bool planned;
    if ((rc = resolve_row_part(ctx, part0, &row_part, B, &planned)) != CFGZIP_OK) return rc;
    PlanUse plan_use(ctx, planned);
    PartSet ps;
    const bool mixed = row_part != nullptr;
    if ((rc = resolve_parts(ctx, part0, mixed, &ps)) != CFGZIP_OK) return rc;
    if (B == 0) return CFGZIP_OK;
    if (!vocab_mask || vocab_stride_words < ps.VW || class_stride_words < ps.maxKW) return CFGZIP_E_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    StepArgs a{};
    a.parts = ctx->d_parts;
    a.part0 = part0;
    a.n_parts = int32_t(ctx->parts.size());
    a.row_part = row_part;
    a.class_mask = class_mask;
    a.cm_stride = class_stride_words;
    a.vocab_mask = vocab_mask;
    a.vm_stride = vocab_stride_words;
    a.B = B;
    a.V = ps.V;
    a.VW = ps.VW;
    a.partials = ctx->d_partials;
    a.tickets = ctx->d_tickets;
    a.status = ctx->d_status;
    a.scale = kLog2e;
    a.inv_t = 1.f;
    if (mode == CFGZIP_SPARSE) {
        int S, per_split;
        if (plan_sparse(ctx, ps, B, false, &S, &per_split)) {
            a.S = S;
            a.per_split = per_split;
            const size_t smem = size_t(per_split) * 4;
            auto kern = k_step_sparse<kF32, false>;
            if ((rc = ensure_smem(kern, smem)) != CFGZIP_OK) return rc;
            return launch(ctx, kern, dim3(unsigned(B) * unsigned(S)), dim3(256), smem, st, a);
        }
        return launch(ctx, k_step_generic<kF32, false>, dim3(unsigned(B)), dim3(256), 0, st, a);
    }
    const DensePlan d = plan_dense(ctx, ps, B, mixed, ps.VW, 8, false);
    if (!d.ok) return launch(ctx, k_step_generic<kF32, false>, dim3(unsigned(B)), dim3(256), 0, st, a);
    if (d.use_plan_kernel && (rc = run_plan_kernel(ctx, row_part, B, ps.V, d, st)) != CFGZIP_OK) return rc;
    fill_groups(ctx, a, d);
    if ((rc = ensure_smem(k_expand_dense, d.smem)) != CFGZIP_OK) return rc;
    return launch(ctx, k_expand_dense, dim3(unsigned(d.n_groups_ub) * unsigned(d.S)), dim3(256), d.smem, st, a);
}

int cfgzip_mask_logits(cfgzip_ctx* ctx, void* logits, int dtype, int64_t row_stride_elems, int32_t B, int32_t V,
                       const uint32_t* vocab_mask, int64_t vocab_stride_words, void* stream) {
    if (!ctx || B < 0 || V <= 0 || (dtype != CFGZIP_F32 && dtype != CFGZIP_BF16)) return CFGZIP_E_ARG;
    if (B == 0) return CFGZIP_OK;
    const int VW = ceil_div(V, 32);
    if (!logits || !vocab_mask || row_stride_elems < V || vocab_stride_words < VW) return CFGZIP_E_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int es = dtype == CFGZIP_BF16 ? 2 : 4;
    const bool al = aligned16(logits, row_stride_elems, es);
    const int n_octets = ceil_div(V, 8);
    const int64_t items = int64_t(B) * ceil_div(n_octets, 256 * 4);
    const unsigned grid = unsigned(std::min<int64_t>(items, int64_t(ctx->sm_count) * 8));
    if (dtype == CFGZIP_BF16) {
        auto kern = al ? k_mask_logits<kBF16, true> : k_mask_logits<kBF16, false>;
        return launch(ctx, kern, dim3(grid), dim3(256), 0, st, logits, row_stride_elems, int(B), int(V), VW, vocab_mask,
                      vocab_stride_words, 0);
    }
    auto kern = al ? k_mask_logits<kF32, true> : k_mask_logits<kF32, false>;
    return launch(ctx, kern, dim3(grid), dim3(256), 0, st, logits, row_stride_elems, int(B), int(V), VW, vocab_mask,
                  vocab_stride_words, aligned32(logits, row_stride_elems, 4) ? 1 : 0);
}

int cfgzip_masked_logsoftmax_argmax(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part,
                                    const uint32_t* class_mask, int64_t class_stride_words, void* logits, int dtype,
                                    int64_t row_stride_elems, int32_t B, uint32_t* vocab_mask,
                                    int64_t vocab_stride_words, int32_t* argmax, int32_t* rep, float* logp_argmax,
                                    float* lse, float* logp_full, int mode, void* stream) {
    int rc = check_step_args(ctx, class_mask, class_stride_words, B, mode);
    if (rc != CFGZIP_OK) return rc;
    if (dtype != CFGZIP_F32 && dtype != CFGZIP_BF16) return CFGZIP_E_ARG;
    bool planned;
    if ((rc = resolve_row_part(ctx, part0, &row_part, B, &planned)) != CFGZIP_OK) return rc;
    PlanUse plan_use(ctx, planned);
    PartSet ps;
    const bool mixed = row_part != nullptr;
    if ((rc = resolve_parts(ctx, part0, mixed, &ps)) != CFGZIP_OK) return rc;
    if (B == 0) return CFGZIP_OK;
    if (!logits || !argmax || row_stride_elems < ps.V || class_stride_words < ps.maxKW) return CFGZIP_E_ARG;
    if (vocab_mask && vocab_stride_words < ps.VW) return CFGZIP_E_ARG;
    if (logp_full && !lse) return CFGZIP_E_ARG;  // the full log-probabilities are formed from lse
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    StepArgs a{};
    a.parts = ctx->d_parts;
    a.part0 = part0;
    a.n_parts = int32_t(ctx->parts.size());
    a.row_part = row_part;
    a.class_mask = class_mask;
    a.cm_stride = class_stride_words;
    a.logits = logits;
    a.row_stride = row_stride_elems;
    a.vocab_mask = vocab_mask;
    a.vm_stride = vocab_stride_words;
    a.argmax = argmax;
    a.rep = rep;
    a.logp_argmax = logp_argmax;
    a.lse = lse;
    a.B = B;
    a.V = ps.V;
    a.VW = ps.VW;
    a.partials = ctx->d_partials;
    a.tickets = ctx->d_tickets;
    a.status = ctx->d_status;
    a.scale = kLog2e;
    a.inv_t = 1.f;
    const int es = dtype == CFGZIP_BF16 ? 2 : 4;
    const bool al = aligned16(logits, row_stride_elems, es);
    a.wide = aligned32(logits, row_stride_elems, es);  // 32-byte stores (f32 octets, bf16 octet pairs)
    // measured: early launch of the next kernel (whose blocks set themselves up meanwhile) helps steps up to
    // about 130 MB of logits (B = 512 bf16: -1.3 %) and costs 1 % and more from 260 MB on
    ctx->pdl_now = int64_t(B) * ps.V * es < (int64_t(192) << 20);
    ctx->prefetch_now = int64_t(B) * ps.V * es >= (int64_t(ctx->prefetch_min_mbytes) << 20);
    rc = dtype == CFGZIP_BF16 ? launch_fused<kBF16>(ctx, a, ps, mixed, mode, al, logp_full, st)
                              : launch_fused<kF32>(ctx, a, ps, mixed, mode, al, logp_full, st);
    ctx->pdl_now = true;
    return rc;
}

int cfgzip_masked_sample(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part, const uint32_t* class_mask,
                         int64_t class_stride_words, void* logits, int dtype, int64_t row_stride_elems, int32_t B,
                         uint32_t* vocab_mask, int64_t vocab_stride_words, const float* u, float inv_temperature,
                         int32_t* token, int32_t* rep, float* logp_token, float* lse, int mode, void* stream) {
    return cfgzip_masked_sample_filtered(ctx, part0, row_part, class_mask, class_stride_words, logits, dtype, row_stride_elems,
                                         B, vocab_mask, vocab_stride_words, u, inv_temperature, 0, 1.f, token, rep, logp_token,
                                         lse, mode, stream);
}

int cfgzip_masked_sample_filtered(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part,
                                  const uint32_t* class_mask, int64_t class_stride_words, void* logits, int dtype,
                                  int64_t row_stride_elems, int32_t B, uint32_t* vocab_mask, int64_t vocab_stride_words,
                                  const float* u, float inv_temperature, int32_t top_k, float top_p, int32_t* token,
                                  int32_t* rep, float* logp_token, float* lse, int mode, void* stream) {
    if (top_k < 0 || !(top_p > 0.f)) return CFGZIP_E_ARG;
    int rc = check_step_args(ctx, class_mask, class_stride_words, B, mode);
    if (rc != CFGZIP_OK) return rc;
    if (dtype != CFGZIP_F32 && dtype != CFGZIP_BF16) return CFGZIP_E_ARG;
    if (mode == CFGZIP_SPARSE) return CFGZIP_E_ARG;  // the class-list kernel does not leave its states in token order
    if (!(inv_temperature > 0.f) || !(inv_temperature <= 1e6f)) return CFGZIP_E_ARG;
    bool planned;
    if ((rc = resolve_row_part(ctx, part0, &row_part, B, &planned)) != CFGZIP_OK) return rc;
    PlanUse plan_use(ctx, planned);
    PartSet ps;
    const bool mixed = row_part != nullptr;
    if ((rc = resolve_parts(ctx, part0, mixed, &ps)) != CFGZIP_OK) return rc;
    if (B == 0) return CFGZIP_OK;
    if (!logits || !token || !u || row_stride_elems < ps.V || class_stride_words < ps.maxKW) return CFGZIP_E_ARG;
    if (vocab_mask && vocab_stride_words < ps.VW) return CFGZIP_E_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    StepArgs a{};
    a.parts = ctx->d_parts;
    a.part0 = part0;
    a.n_parts = int32_t(ctx->parts.size());
    a.row_part = row_part;
    a.class_mask = class_mask;
    a.cm_stride = class_stride_words;
    a.logits = logits;
    a.row_stride = row_stride_elems;
    a.vocab_mask = vocab_mask;
    a.vm_stride = vocab_stride_words;
    a.argmax = token;
    a.rep = rep;
    a.logp_argmax = logp_token;
    a.lse = lse;
    a.B = B;
    a.V = ps.V;
    a.VW = ps.VW;
    a.partials = ctx->d_partials;
    a.tickets = ctx->d_tickets;
    a.status = ctx->d_status;
    a.scale = kLog2e * inv_temperature;
    a.inv_t = inv_temperature;
    a.u = u;
    const int es = dtype == CFGZIP_BF16 ? 2 : 4;
    const bool al = aligned16(logits, row_stride_elems, es);
    a.wide = aligned32(logits, row_stride_elems, es);
    ctx->pdl_now = int64_t(B) * ps.V * es < (int64_t(192) << 20);
    ctx->prefetch_now = int64_t(B) * ps.V * es >= (int64_t(ctx->prefetch_min_mbytes) << 20);
    rc = dtype == CFGZIP_BF16 ? launch_sample<kBF16>(ctx, a, ps, mixed, al, top_k, top_p, st)
                              : launch_sample<kF32>(ctx, a, ps, mixed, al, top_k, top_p, st);
    ctx->pdl_now = true;
    return rc;
}

int cfgzip_multi_mask_logsoftmax_argmax(cfgzip_ctx* ctx, cfgzip_part_id part0, const uint32_t* class_masks,
                                        int64_t class_stride_words, int32_t masks_per_row, const void* logits, int dtype,
                                        int64_t row_stride_elems, int32_t B, uint32_t* vocab_masks,
                                        int64_t vocab_stride_words, int32_t* argmax, int32_t* rep, float* logp_argmax,
                                        float* lse, void* stream) {
    if (!ctx || B < 0 || masks_per_row < 1 || (dtype != CFGZIP_F32 && dtype != CFGZIP_BF16)) return CFGZIP_E_ARG;
    PartSet ps;
    int rc = resolve_parts(ctx, part0, false, &ps);
    if (rc != CFGZIP_OK) return rc;
    if (B == 0) return CFGZIP_OK;
    if (int64_t(B) * masks_per_row > ctx->reserved_rows) return CFGZIP_E_NOMEM;
    if (!class_masks || !logits || !argmax || class_stride_words < ps.maxKW || row_stride_elems < ps.V) return CFGZIP_E_ARG;
    if (vocab_masks && vocab_stride_words < ps.VW) return CFGZIP_E_ARG;
    const int es = dtype == CFGZIP_BF16 ? 2 : 4;
    if (!aligned16(logits, row_stride_elems, es)) return CFGZIP_E_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int32_t rows = B * masks_per_row;  // one "row" of masks, vocab masks and results per (logits row, mask)
    StepArgs a{};
    a.parts = ctx->d_parts;
    a.part0 = part0;
    a.n_parts = int32_t(ctx->parts.size());
    a.class_mask = class_masks;
    a.cm_stride = class_stride_words;
    a.logits = const_cast<void*>(logits);  // never written: masks_per_row > 0 switches the write-back off
    a.row_stride = row_stride_elems;
    a.vocab_mask = vocab_masks;
    a.vm_stride = vocab_stride_words;
    a.argmax = argmax;
    a.rep = rep;
    a.logp_argmax = logp_argmax;
    a.lse = lse;
    a.B = rows;
    a.V = ps.V;
    a.VW = ps.VW;
    a.partials = ctx->d_partials;
    a.tickets = ctx->d_tickets;
    a.status = ctx->d_status;
    a.scale = kLog2e;
    a.inv_t = 1.f;
    a.masks_per_row = masks_per_row;
    const DensePlan d = plan_dense(ctx, ps, rows, false, 4 * ps.VW, 32, true);
    if (!d.ok) return CFGZIP_E_RANGE;  // more than 65535 classes, or a class table beyond shared memory
    fill_groups(ctx, a, d);
    ctx->pdl_now = int64_t(B) * ps.V * es < (int64_t(192) << 20);
    ctx->prefetch_now = int64_t(B) * ps.V * es >= (int64_t(ctx->prefetch_min_mbytes) << 20);
    auto kern = dtype == CFGZIP_BF16 ? k_step_dense<kBF16> : k_step_dense<kF32>;
    if ((rc = ensure_smem(kern, d.smem)) == CFGZIP_OK)
        rc = launch(ctx, kern, dim3(unsigned(d.n_groups_ub) * unsigned(d.S)), dim3(unsigned(d.threads)), d.smem, st, a);
    if (rc == CFGZIP_OK) {
        auto fin = dtype == CFGZIP_BF16 ? k_finalize_rows<kBF16> : k_finalize_rows<kF32>;
        rc = launch(ctx, fin, dim3(unsigned(d.n_groups_ub) * kGroupRows), dim3(kFinalizeThreads), 0, st, a);
    }
    ctx->pdl_now = true;
    return rc;
}

int cfgzip_plan_rows(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part, int32_t B, void* stream) {
    if (!ctx || !row_part || row_part == CFGZIP_ROWS_AS_PLANNED || B <= 0) return CFGZIP_E_ARG;
    PartSet ps;
    int rc = resolve_parts(ctx, part0, true, &ps);
    if (rc != CFGZIP_OK) return rc;
    if (B > ctx->reserved_rows) return CFGZIP_E_NOMEM;
    DensePlan d;
    d.n_groups_ub = ceil_div(B, kGroupRows) + ps.n_live_same_v;
    if (d.n_groups_ub > ctx->max_groups) return CFGZIP_E_NOMEM;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    ctx->plan_in_use = false;
    if ((rc = run_plan_kernel(ctx, row_part, B, ps.V, d, static_cast<cudaStream_t>(stream))) != CFGZIP_OK) return rc;
    ctx->plan_valid = true;
    ctx->plan_row_part = row_part;
    ctx->plan_B = B;
    ctx->plan_V = ps.V;
    return CFGZIP_OK;
}

int cfgzip_map_tokens(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part, const int32_t* tokens,
                      int32_t* reps, int32_t B, void* stream) {
    if (!ctx || B < 0) return CFGZIP_E_ARG;
    bool planned;
    int rc = resolve_row_part(ctx, part0, &row_part, B, &planned);
    if (rc != CFGZIP_OK) return rc;
    PartSet ps;
    rc = resolve_parts(ctx, part0, row_part != nullptr, &ps);
    if (rc != CFGZIP_OK) return rc;
    if (B == 0) return CFGZIP_OK;
    if (!tokens || !reps) return CFGZIP_E_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    return launch(ctx, k_map_tokens, dim3(unsigned(ceil_div(B, 256))), dim3(256), 0, static_cast<cudaStream_t>(stream),
                  (const PartDev*)ctx->d_parts, int(ctx->parts.size()), int(part0), row_part, tokens, reps, int(B),
                  int(ps.V), ctx->d_status);
}

int cfgzip_choose_mode(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part_host,
                       const uint32_t* class_mask_host, int64_t class_stride_words, int32_t B, int dtype) {
    if (!ctx || B < 0 || (dtype != CFGZIP_F32 && dtype != CFGZIP_BF16)) return CFGZIP_E_ARG;
    if (row_part_host == CFGZIP_ROWS_AS_PLANNED) return CFGZIP_E_ARG;
    PartSet ps;
    int rc = resolve_parts(ctx, part0, row_part_host != nullptr, &ps);
    if (rc != CFGZIP_OK) return rc;
    if (B == 0) return CFGZIP_DENSE;
    if (!class_mask_host || class_stride_words < ps.maxKW) return CFGZIP_E_ARG;
    const int permille = ctx->auto_permille >= 0 ? ctx->auto_permille : (dtype == CFGZIP_BF16 ? 10 : 40);
    // the gather kernel wins as soon as the allowed tokens reach permille / 1000 of the batch (rows with a bad partition
    // id count as rows: they make the batch look sparser, never denser): stop counting there
    const unsigned long long enough = (static_cast<unsigned long long>(permille) * unsigned(B) * unsigned(ps.V) + 999ull) / 1000ull;
    unsigned long long allowed = 0;
    for (int32_t b = 0; b < B && allowed < enough; ++b) {
        const int32_t id = row_part_host ? row_part_host[b] : part0;
        if (id < 0 || size_t(id) >= ctx->parts.size() || !ctx->parts[size_t(id)].live || ctx->parts[size_t(id)].V != ps.V) continue;
        const Part& p = ctx->parts[size_t(id)];
        const uint32_t* m = class_mask_host + int64_t(b) * class_stride_words;
        for (int32_t kw = 0; kw < p.KW; ++kw) {
            uint32_t word = m[kw];
            if (kw == p.KW - 1 && (p.K & 31)) word &= (1u << (p.K & 31)) - 1u;
            while (word) {
                allowed += unsigned(p.sizes[size_t(kw) * 32 + size_t(__builtin_ctz(word))]);
                word &= word - 1u;
            }
        }
    }
    return allowed * 1000ull < static_cast<unsigned long long>(permille) * unsigned(B) * unsigned(ps.V) ? CFGZIP_SPARSE : CFGZIP_DENSE;
}

int cfgzip_decode_step_host(cfgzip_ctx* ctx, cfgzip_part_id part0, const int32_t* row_part_host,
                            const uint32_t* class_mask_host, int64_t class_stride_words, const void* logits_host,
                            int dtype, int32_t B, void* masked_logits, uint32_t* vocab_mask_host, int32_t* argmax,
                            int32_t* rep, float* logp_argmax, float* lse, int mode, void* stream) {
    int rc = check_step_args(ctx, class_mask_host, class_stride_words, B, mode);
    if (rc != CFGZIP_OK) return rc;
    if (dtype != CFGZIP_F32 && dtype != CFGZIP_BF16) return CFGZIP_E_ARG;
    if (row_part_host == CFGZIP_ROWS_AS_PLANNED) return CFGZIP_E_ARG;  // a kept grouping refers to a device vector
    PartSet ps;
    if ((rc = resolve_parts(ctx, part0, row_part_host != nullptr, &ps)) != CFGZIP_OK) return rc;
    if (B == 0) return CFGZIP_OK;
    if (!logits_host || class_stride_words < ps.maxKW) return CFGZIP_E_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t es = dtype == CFGZIP_BF16 ? 2 : 4;
    const size_t logit_bytes = size_t(B) * size_t(ps.V) * es;
    const size_t cm_bytes = size_t(B) * size_t(class_stride_words) * 4;
    const size_t vm_bytes = size_t(B) * size_t(ps.VW) * 4;
    if (logit_bytes > ctx->st_logits_bytes || cm_bytes > ctx->st_cm_bytes || vm_bytes > ctx->st_vm_bytes ||
        B > ctx->st_rows) {
        cudaStreamSynchronize(st);
        if ((rc = grow(&ctx->st_logits, &ctx->st_logits_bytes, logit_bytes)) != CFGZIP_OK) return rc;
        if ((rc = grow(reinterpret_cast<void**>(&ctx->st_cm), &ctx->st_cm_bytes, cm_bytes)) != CFGZIP_OK) return rc;
        if ((rc = grow(reinterpret_cast<void**>(&ctx->st_vm), &ctx->st_vm_bytes, vm_bytes)) != CFGZIP_OK) return rc;
        if (B > ctx->st_rows) {
            size_t have = size_t(ctx->st_rows) * 20;
            if ((rc = grow(reinterpret_cast<void**>(&ctx->st_small), &have, size_t(B) * 20)) != CFGZIP_OK) {
                ctx->st_rows = 0;
                return rc;
            }
            ctx->st_rows = B;
            if (ctx->st_small_host) cudaFreeHost(ctx->st_small_host);
            ctx->st_small_host = nullptr;
            if (cudaHostAlloc(reinterpret_cast<void**>(&ctx->st_small_host), size_t(B) * 16, cudaHostAllocDefault) != cudaSuccess) {
                cudaGetLastError();
                ctx->st_small_host = nullptr;  // the four results then come back one by one
            }
        }
    }
    int32_t* d_rp = ctx->st_small;
    int32_t* d_am = d_rp + ctx->st_rows;
    int32_t* d_rep = d_am + ctx->st_rows;
    float* d_lse = reinterpret_cast<float*>(d_rep + ctx->st_rows);
    float* d_lpa = d_lse + ctx->st_rows;
    bool ok = cudaMemcpyAsync(ctx->st_cm, class_mask_host, cm_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaMemcpyAsync(ctx->st_logits, logits_host, logit_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (ok && row_part_host)
        ok = cudaMemcpyAsync(d_rp, row_part_host, size_t(B) * 4, cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        return CFGZIP_E_CUDA;
    }
    if (mode == CFGZIP_AUTO) {  // the class masks are in host memory: the choice costs no launch
        const int chosen = cfgzip_choose_mode(ctx, part0, row_part_host, class_mask_host, class_stride_words, B, dtype);
        if (chosen > 0) mode = chosen;
    }
    rc = cfgzip_masked_logsoftmax_argmax(ctx, part0, row_part_host ? d_rp : nullptr, ctx->st_cm, class_stride_words,
                                         ctx->st_logits, dtype, ps.V, B, vocab_mask_host ? ctx->st_vm : nullptr, ps.VW,
                                         d_am, d_rep, d_lpa, d_lse, nullptr, mode, stream);
    if (rc != CFGZIP_OK) return rc;
    auto back = [&](void* dst, const void* src, size_t n) {
        if (dst && ok) ok = cudaMemcpyAsync(dst, src, n, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    };
    back(masked_logits, ctx->st_logits, logit_bytes);
    back(vocab_mask_host, ctx->st_vm, vm_bytes);
    // the four small result arrays sit side by side on the device: one copy into a pinned mirror, handed out
    // after the stream has drained (four separate small copies cost more than the kernels of a short step)
    const bool one_copy = ctx->st_small_host != nullptr && (argmax || rep || lse || logp_argmax);
    const size_t span = (size_t(ctx->st_rows) * 3 + size_t(B)) * 4;  // argmax .. logp_argmax, st_rows apart
    if (one_copy) {
        back(ctx->st_small_host, d_am, span);
    } else {
        back(argmax, d_am, size_t(B) * 4);
        back(rep, d_rep, size_t(B) * 4);
        back(lse, d_lse, size_t(B) * 4);
        back(logp_argmax, d_lpa, size_t(B) * 4);
    }
    if (!ok || cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return CFGZIP_E_CUDA;
    }
    if (one_copy) {
        const int32_t* h = ctx->st_small_host;
        const size_t n = size_t(B) * 4, step = size_t(ctx->st_rows);
        if (argmax) std::memcpy(argmax, h, n);
        if (rep) std::memcpy(rep, h + step, n);
        if (lse) std::memcpy(lse, h + 2 * step, n);
        if (logp_argmax) std::memcpy(logp_argmax, h + 3 * step, n);
    }
    return CFGZIP_OK;
}

int cfgzip_poll_status(cfgzip_ctx* ctx, void* stream, int32_t* n_empty_rows, int32_t* n_bad_tokens,
                       int32_t* n_bad_rows) {
    if (!ctx) return CFGZIP_E_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t h[4] = {0, 0, 0, 0};
    if (cudaMemcpyAsync(h, ctx->d_status, sizeof h, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemsetAsync(ctx->d_status, 0, sizeof h, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return CFGZIP_E_CUDA;
    }
    if (n_empty_rows) *n_empty_rows = h[0];
    if (n_bad_tokens) *n_bad_tokens = h[1];
    if (n_bad_rows) *n_bad_rows = h[2];
    return h[3] ? CFGZIP_E_CUDA : CFGZIP_OK;  // h[3]: asynchronous copies that never completed
}

int cfgzip_rmw_floor(cfgzip_ctx* ctx, void* logits, int dtype, int64_t row_stride_elems, int32_t B, int32_t V,
                     void* stream) {
    if (!ctx || B < 0 || V <= 0 || (dtype != CFGZIP_F32 && dtype != CFGZIP_BF16)) return CFGZIP_E_ARG;
    if (B == 0) return CFGZIP_OK;
    if (!logits || row_stride_elems < V) return CFGZIP_E_ARG;
    const int es = dtype == CFGZIP_BF16 ? 2 : 4;
    if (!aligned16(logits, row_stride_elems, es)) return CFGZIP_E_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return CFGZIP_E_CUDA;
    const int64_t items = int64_t(B) * ceil_div((int64_t(V) * es) >> 4, 256 * 4);
    if (items == 0) return CFGZIP_OK;
    const unsigned grid = unsigned(std::min<int64_t>(items, int64_t(ctx->sm_count) * 8));
    ctx->pdl_now = int64_t(B) * V * es < (int64_t(192) << 20);
    ctx->prefetch_now = int64_t(B) * V * es >= (int64_t(ctx->prefetch_min_mbytes) << 20);
    const int rc = dtype == CFGZIP_BF16
                       ? launch(ctx, k_rmw_floor<kBF16>, dim3(grid), dim3(256), 0, static_cast<cudaStream_t>(stream), logits,
                                row_stride_elems, int(B), int(V))
                       : launch(ctx, k_rmw_floor<kF32>, dim3(grid), dim3(256), 0, static_cast<cudaStream_t>(stream), logits,
                                row_stride_elems, int(B), int(V));
    ctx->pdl_now = true;
    return rc;
}

int cfgzip_launch_count(cfgzip_ctx* ctx, int64_t* out) {
    if (!ctx || !out) return CFGZIP_E_ARG;
    *out = ctx->launches;
    return CFGZIP_OK;
}

int cfgzip_set_tuning(cfgzip_ctx* ctx, const char* name, int32_t value) {
    if (!ctx || !name) return CFGZIP_E_ARG;
    if (!std::strcmp(name, "ctas_per_sm")) {
        if (value < 1 || value > 16) return CFGZIP_E_ARG;
        ctx->ctas_per_sm = value;
    } else if (!std::strcmp(name, "token_warps")) {
        if (value < 0 || value > 16) return CFGZIP_E_ARG;
        ctx->token_warps = value;
    } else if (!std::strcmp(name, "row_warps")) {
        if (value != 0 && value != 1 && value != 2 && value != 4) return CFGZIP_E_ARG;
        ctx->row_warps = value;
    } else if (!std::strcmp(name, "pdl")) {
        if (value < 0 || value > 2) return CFGZIP_E_ARG;
        ctx->pdl = value;
    } else if (!std::strcmp(name, "pipeline")) {
        ctx->pipeline = value ? 1 : 0;
    } else if (!std::strcmp(name, "tensor_map")) {
        ctx->tensor_map = value ? 1 : 0;
    } else if (!std::strcmp(name, "pipe_warps")) {
        if (value < 1 || value > 16) return CFGZIP_E_ARG;
        ctx->pipe_warps = value;
    } else if (!std::strcmp(name, "waves")) {
        if (value < 1 || value > 16) return CFGZIP_E_ARG;
        ctx->waves = value;
    } else if (!std::strcmp(name, "spread")) {
        ctx->spread = value ? 1 : 0;
    } else if (!std::strcmp(name, "stage_alias")) {
        ctx->stage_alias = value ? 1 : 0;
    } else if (!std::strcmp(name, "auto_sparse_permille")) {
        if (value < -1 || value > 1000) return CFGZIP_E_ARG;
        ctx->auto_permille = value;
    } else if (!std::strcmp(name, "auto_min_mbytes")) {
        if (value < -1) return CFGZIP_E_ARG;
        ctx->auto_min_bytes = value < 0 ? -1 : int64_t(value) << 20;
    } else if (!std::strcmp(name, "prefetch_items")) {
        if (value < 0 || value > 64) return CFGZIP_E_ARG;
        ctx->prefetch_items = value;
    } else if (!std::strcmp(name, "prefetch_min_mbytes")) {
        if (value < 0) return CFGZIP_E_ARG;
        ctx->prefetch_min_mbytes = value;
    } else if (!std::strcmp(name, "rotate")) {
        ctx->rotate = value != 0;
    } else if (!std::strcmp(name, "fold")) {
        if (value < 0 || value > 2) return CFGZIP_E_ARG;
        ctx->fold = value;
    } else if (!std::strcmp(name, "lane_octets")) {
        if (value < 0 || value > 2) return CFGZIP_E_ARG;
        ctx->lane_octets = value;
    } else if (!std::strcmp(name, "test_expire_waits")) {
        ctx->expire_test = value ? 1 : 0;
    } else if (!std::strcmp(name, "pipe_depth")) {
        if (value < 2 || value > 8) return CFGZIP_E_ARG;
        ctx->pipe_depth = value;
        ctx->pipe_depth_set = true;
    } else {
        return CFGZIP_E_ARG;
    }
    return CFGZIP_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// cfgzip_step_noalloc: see include/cfgzip.h. In host code `g_noalloc_scratch` is only a handle
// for the runtime; the device address of each GPU's copy is asked for once per device.
// ---------------------------------------------------------------------------------------------
namespace {
constexpr int kMaxDevices = 64;
struct NoAllocDevice {
    NoAllocScratch* scratch = nullptr;
    int sm_count = 0;
};
NoAllocDevice g_noalloc_dev[kMaxDevices];
std::mutex g_noalloc_mutex;
}  // namespace

extern "C" int cfgzip_step_noalloc(const int32_t* token_to_class, int32_t V, const int32_t* class_to_rep, int32_t K,
                                   const uint32_t* class_mask, int64_t class_stride_words, void* logits, int dtype,
                                   int64_t row_stride_elems, int32_t B, uint32_t* vocab_mask, int64_t vocab_stride_words,
                                   int32_t* argmax, int32_t* rep, float* logp_argmax, float* lse, void* stream) {
    if (V <= 0 || K <= 0 || K > V || B < 0 || (dtype != CFGZIP_F32 && dtype != CFGZIP_BF16)) return CFGZIP_E_ARG;
    if (B == 0) return CFGZIP_OK;
    if (B > kNoAllocMaxRows) return CFGZIP_E_RANGE;  // more rows than the built-in scratch has tickets for
    const int VW = ceil_div(V, 32), KW = ceil_div(K, 32);
    if (!token_to_class || !class_to_rep || !class_mask || !logits || !argmax) return CFGZIP_E_ARG;
    if (class_stride_words < KW || row_stride_elems < V || (vocab_mask && vocab_stride_words < VW)) return CFGZIP_E_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return CFGZIP_E_CUDA;
    }
    NoAllocDevice nd;
    {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_dev[dev].scratch) {
            // first call on this GPU (it is the current device): ask where its copy of the array lives
            NoAllocScratch* ptr = nullptr;
            int sms = 0;
            if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch) != cudaSuccess || !ptr ||
                cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
                cudaGetLastError();
                return CFGZIP_E_CUDA;
            }
            g_noalloc_dev[dev].scratch = ptr;
            g_noalloc_dev[dev].sm_count = sms;
        }
        nd = g_noalloc_dev[dev];
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the last call left: the tickets must read zero when the kernel starts
    if (cudaMemsetAsync(nd.scratch->tickets, 0, sizeof(unsigned int) * size_t(B), st) != cudaSuccess) {
        cudaGetLastError();
        return CFGZIP_E_CUDA;
    }
    RowSplitArgs a{};
    a.c = token_to_class;
    a.r = class_to_rep;
    a.V = V;
    a.K = K;
    a.VW = VW;
    a.class_mask = class_mask;
    a.cm_stride = class_stride_words;
    a.logits = logits;
    a.row_stride = row_stride_elems;
    a.vocab_mask = vocab_mask;
    a.vm_stride = vocab_stride_words;
    a.argmax = argmax;
    a.rep = rep;
    a.logp_argmax = logp_argmax;
    a.lse = lse;
    a.B = B;
    int S = std::max(1, (4 * nd.sm_count) / B);
    S = std::min(S, std::min(kNoAllocMaxSplits, std::max(1, VW / 64)));
    a.words_per_split = ceil_div(VW, S);
    a.S = ceil_div(VW, a.words_per_split);
    a.partials = nd.scratch->partials;
    a.tickets = nd.scratch->tickets;
    const dim3 grid(unsigned(B) * unsigned(a.S)), block(256);
    if (dtype == CFGZIP_BF16)
        k_step_rowsplit<kBF16><<<grid, block, 0, st>>>(a);
    else
        k_step_rowsplit<kF32><<<grid, block, 0, st>>>(a);
    if (cudaGetLastError() != cudaSuccess) return CFGZIP_E_CUDA;
    return CFGZIP_OK;
}

// ---------------------------------------------------------------------------------------------
// Host-only view of the launch planner, for tests: no GPU is touched. See include/cfgzip.h.
// ---------------------------------------------------------------------------------------------
extern "C" int cfgzip_plan_query(int32_t sm_count, int32_t smem_optin, int32_t V, int32_t K, int32_t B, int dtype,
                                 int32_t n_partitions, int32_t aligned_class_masks, int32_t out[16]) {
    if (!out || sm_count <= 0 || smem_optin <= 0 || V <= 0 || K <= 0 || K > V || B <= 0 || n_partitions <= 0 ||
        (dtype != CFGZIP_F32 && dtype != CFGZIP_BF16))
        return CFGZIP_E_ARG;
    cfgzip_ctx fake;  // plain host object: the planners read its limits and tuning fields only
    fake.sm_count = sm_count;
    fake.smem_optin = smem_optin;
    fake.reserved_rows = kDefaultRows;
    fake.max_groups = ceil_div(kDefaultRows, kGroupRows) + kMaxParts;
    PartSet ps;
    ps.V = V;
    ps.VW = ceil_div(V, 32);
    ps.maxK = K;
    ps.maxKW = ceil_div(K, 32);
    ps.n_live_same_v = n_partitions;
    ps.all_c16 = K <= 65535;
    ps.all_kw_mult4 = (ps.maxKW % 4) == 0;
    const bool mixed = n_partitions > 1;
    const int es = dtype == CFGZIP_BF16 ? 2 : 4;
    DensePlan d = plan_pipe(&fake, ps, B, mixed, es, aligned_class_masks != 0);
    int kind = 2;  // pipelined
    if (!d.ok) {
        d = plan_dense(&fake, ps, B, mixed, 4 * ps.VW, 32, true);
        kind = 1;  // register kernel
    }
    if (!d.ok) kind = 0;  // per-row kernel
    int sp_S = 0, sp_per = 0;
    const bool sparse_ok = plan_sparse(&fake, ps, B, true, &sp_S, &sp_per);
    const int32_t vals[16] = {kind, d.n_groups_ub, d.S, d.per_split, d.WT, d.threads, d.depth, int32_t(d.smem),
                              d.table_words, d.stage_stride, d.cm_bulk, d.slots, sparse_ok ? sp_S : 0,
                              sparse_ok ? sp_per : 0, int32_t(kPartialSlots), d.ctas_per_sm};
    std::memcpy(out, vals, sizeof vals);
    return CFGZIP_OK;
}
