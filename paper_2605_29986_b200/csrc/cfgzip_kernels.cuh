// Kernels of the decode-step path. All of them are bandwidth- or latency-bound
// scans: no tensor cores. Notation: V tokens, K classes, B rows, VW = ceil(V/32),
// KW = ceil(K/32); an "octet" is 8 consecutive tokens of one row (16 bytes of bf16,
// 32 bytes of f32, one byte of vocab mask).
#pragma once

#include <cuda.h>
#include <type_traits>

#include "cfgzip_device.cuh"

namespace cfgzip {

// Arguments of one step (expand / fused), shared by the dense, sparse and generic kernels.
struct StepArgs {
    const PartDev* parts;
    int32_t part0;
    int32_t n_parts;
    const int32_t* row_part;    // dev [B] or null
    // row groups (dense kernels): null = implicit groups of 32 consecutive rows using part0
    const int32_t* group_part;  // dev [n_groups]
    const int32_t* group_rows;  // dev [n_groups * 32], -1 = empty slot, valid slots first
    const int32_t* n_groups;    // dev scalar
    const uint32_t* class_mask;
    int64_t cm_stride;
    void* logits;
    int64_t row_stride;         // elements
    uint32_t* vocab_mask;       // nullable
    int64_t vm_stride;
    int32_t* argmax;
    int32_t* rep;
    float* logp_argmax;
    float* lse;
    int32_t B, V, VW;
    int32_t S;                  // CTAs that share one group (dense) or one row (sparse)
    int32_t slots;              // dense: published states per row (S * WT + 1)
    int32_t per_split;          // octets (dense) or vocab-mask words (sparse) per CTA
    int32_t WT;                 // dense: warps side by side along the vocabulary
    int32_t table_words;        // dense: shared-memory words of the bit-sliced class table
    int32_t stage_stride;       // dense: words per row of the class-mask staging area, 0 = no staging
    int32_t depth;              // pipelined dense kernel: stages per warp
    int32_t cm_bulk;            // pipelined dense kernel: class-mask rows are fetched by bulk copies (16-byte aligned rows)
    int32_t wide;               // every row of the logits starts on a 32-byte boundary: f32 octets go back as one 32-byte store
    int32_t stage_alias;        // pipelined dense kernel: the class-mask staging area lies over the start of the rings
    int32_t hold_warps;         // stage_alias: warps whose ring it covers; they start their copies after the table is built
    int32_t run_chunks;         // sampling step: every warp slot of the pipelined kernel takes one contiguous run of this
                                // many chunks, so that the published states of a row follow the token order
    int32_t chunk_tokens;       // tokens of one chunk of the pipelined kernel (256 or 512): sampling kernel's run length unit
    int32_t prefetch_items;     // pipelined kernel without a row plan: work items per warp whose logits are asked into the L2
                                // before the wait for the kernel in front (a hint; nothing is read until after the wait)
    int32_t rot_chunks;         // pipelined kernel, greedy step: the round-robin deal of a row batch's chunks starts this many
                                // warp slots further on for every next row batch of the group
    int32_t expire_test;        // test hook: the pipelined kernel reports its first completed wait as run out
    int32_t fold;               // pipelined kernel: the last block of a row group folds the group's states and writes the
                                // rows' results itself (no second kernel); tickets[g] counts the group's finished blocks
    int32_t fold_off;           // fold: byte offset, in dynamic shared memory, of the block's own (row, warp) states, which
                                // are merged to one state per row before they are published; 0 = warps publish directly
    int32_t* row_mode;          // automatic mode: dev [B], written by the class-list kernel, which runs first (1 = the row
                                // allowed so few tokens that that kernel finished it), read by the kernels after it; else null
    int32_t auto_permille;      // automatic mode: a row stays with the class lists when under this many thousandths of its tokens are allowed
    int32_t masks_per_row;      // > 0: several class masks per logits row (register dense kernel only): row r of the masks,
                                // vocab masks and results belongs to logits row r / masks_per_row, and the logits are not modified
    int32_t tail_state;         // sampling kernel: the last state of a row stands for the octets past the last whole vector
    float scale;                // log2(e) / temperature: the sums are of exp(z / T); log2(e) in a greedy step
    float inv_t;                // 1 / temperature
    const float* u;             // sampling step: dev [B] uniform numbers in [0, 1), else null
    PartDev p0;                 // descriptor of part0 (saves a dependent load when rows do not mix partitions)
    Partial* partials;
    unsigned int* tickets;
    int32_t* status;            // [0] empty rows, [1] bad tokens, [2] bad rows, [3] copies that never arrived
};

// The logits row behind row r of the masks and results (they differ when a logits row has several masks).
__device__ __forceinline__ int64_t logits_row(const StepArgs& a, int r) { return a.masks_per_row > 0 ? r / a.masks_per_row : r; }

// The two halves separately, for a kernel that sets itself up (nothing read from memory) while the kernel in
// front of it is still running and only then waits for it.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void pdl_prologue() {
    // Let the next kernel of the stream start its launch early, then wait until everything
    // launched before this kernel has completed. Both are no-ops without the launch attribute.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <int DT>
__device__ __forceinline__ float ldcg_elem(const void* base, int64_t idx) {
    if (DT == kBF16) return __uint_as_float(uint32_t(__ldcg(reinterpret_cast<const unsigned short*>(base) + idx)) << 16);
    return __ldcg(reinterpret_cast<const float*>(base) + idx);
}

// Turn a merged row state into the row's outputs. `pos` is an octet index (pos_is_token
// false: the first allowed token of that octet whose value equals m is the choice) or the
// token index itself.
template <int DT>
__device__ void finalize_row(const StepArgs& a, const PartDev& P, int row, float m, float s, int pos,
                             bool pos_is_token) {
    if (row < 0) return;
    int tok = -1, repv = -1;
    float lsev = -INFINITY, lpa = -INFINITY;
    if (pos != kNoPos) {
        if (pos_is_token) {
            tok = pos;
        } else {
            const uint32_t* cm = a.class_mask + int64_t(row) * a.cm_stride;
            const void* base = reinterpret_cast<const char*>(a.logits) + int64_t(row) * a.row_stride * (DT == kBF16 ? 2 : 4);
            for (int j = 0; j < 8 && tok < 0; ++j) {
                const int t = 8 * pos + j;
                if (t >= a.V) break;
                const int k = P.c32[t];
                if (((cm[k >> 5] >> (k & 31)) & 1u) && ldcg_elem<DT>(base, t) == m) tok = t;
            }
        }
        if (tok >= 0) repv = P.trep[tok];
        if (m > kRefFloor && s > 0.f) {
            const float l = logf(s);
            lsev = m + l;
            lpa = -l;
        }
    } else {
        atomicAdd(a.status + 0, 1);
    }
    a.argmax[row] = tok;
    if (a.rep) a.rep[row] = repv;
    if (a.lse) a.lse[row] = lsev;
    if (a.logp_argmax) a.logp_argmax[row] = lpa;
}

// Same for a whole warp whose lanes all hold the row's merged state (octet position): lanes
// 0..15 test the 16 tokens from the winning octet on side by side. A row without a position either
// allows nothing or holds only -inf at its allowed tokens: the class lists give its lowest
// allowed token. Needs first_allowed_share / write_row_outputs (defined below).
template <int DT>
__device__ __forceinline__ void warp_finalize_row(const StepArgs& a, const PartDev& P, int row, float m, float s,
                                                  int pos, int lane);

// Eight tokens handled one element at a time: ragged tail of a row, or unaligned logits.
template <int DT>
__device__ __forceinline__ void octet_scalar(void* row_base, int o, int V, uint32_t byte, float (&f)[8]) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int t = 8 * o + j;
        f[j] = -INFINITY;
        if (t < V) {
            if ((byte >> j) & 1u)
                f[j] = load_elem<DT>(row_base, t);
            else
                store_neg_inf<DT>(row_base, t);
        }
    }
}

// Fill the 32 row slots of group g and return the partition the group uses.
__device__ __forceinline__ int group_rows_setup(const StepArgs& a, int g, int* s_row, int tid) {
    if (tid < kGroupRows) {
        int row;
        if (a.group_rows) {
            row = a.group_rows[g * kGroupRows + tid];
        } else {
            row = g * kGroupRows + tid;
            if (row >= a.B) row = -1;
        }
        s_row[tid] = row;
    }
    return a.group_part ? a.group_part[g] : a.part0;
}

// Copy the class-mask rows of the group's 32 row slots to shared memory (`stage`, rows
// stage_stride words apart). A warp takes one row at a time with coalesced loads, four rows
// and two 32-word spans per pass, so up to eight loads per thread are in flight together.
__device__ __forceinline__ void stage_class_masks(const StepArgs& a, const PartDev& P, const int* s_row, uint32_t* stage,
                                                  int warp, int lane, int n_warps) {
    for (int r0 = warp; r0 < kGroupRows; r0 += 4 * n_warps) {
        for (int kw0 = lane; kw0 < P.KW; kw0 += 64) {
            uint32_t v[4][2];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = r0 + q * n_warps;
                const int row = r < kGroupRows ? s_row[r] : -1;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int kw = kw0 + 32 * u;
                    v[q][u] = (row >= 0 && kw < P.KW) ? __ldg(a.class_mask + int64_t(row) * a.cm_stride + kw) : 0u;
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = r0 + q * n_warps;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int kw = kw0 + 32 * u;
                    if (r < kGroupRows && kw < P.KW) stage[r * a.stage_stride + kw] = v[q][u];
                }
            }
        }
    }
}

// Bit-sliced class table of one row group: T[k] bit r = "row slot r allows class k".
// Entries K .. 32*(KW+1)-1 are zero, so the padding class id K looks up "nobody".
// With a staging area (filled by stage_class_masks, then a block barrier) the 32x32 bit
// blocks are read from shared memory; stage_stride is odd, so those column reads hit 32
// banks. Without one, each lane reads its row's words from global memory, eight at a time.
__device__ __forceinline__ void build_class_table(const StepArgs& a, const PartDev& P, const int* s_row, uint32_t* T,
                                                  const uint32_t* stage, int warp, int lane, int n_warps) {
    const uint32_t tail = (P.K & 31) ? (1u << (P.K & 31)) - 1u : 0xFFFFFFFFu;
    const int row = s_row[lane];
    const uint32_t* cm = a.class_mask + int64_t(row < 0 ? 0 : row) * a.cm_stride;
    constexpr int U = 4;
    for (int kw0 = warp; kw0 <= P.KW; kw0 += n_warps * U) {
        uint32_t x[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int kw = kw0 + u * n_warps;
            x[u] = 0u;
            if (kw < P.KW && row >= 0) x[u] = a.stage_stride ? stage[lane * a.stage_stride + kw] : __ldg(cm + kw);
            if (kw == P.KW - 1) x[u] &= tail;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int kw = kw0 + u * n_warps;
            const uint32_t t = warp_transpose32(x[u], lane);  // independent chains: their shuffles overlap
            if (kw <= P.KW) T[kw * 32 + lane] = t;
        }
    }
}

// The same table from a staging area whose rows are 16-byte aligned and stage_stride (a
// multiple of 4, with stage_stride/4 odd) words apart: a lane reads four words of its row at
// once, which spreads the eight lanes of a quarter warp over all 32 banks.
__device__ __forceinline__ void build_class_table_quads(const StepArgs& a, const PartDev& P, const int* s_row, uint32_t* T,
                                                        const uint32_t* stage, int warp, int lane, int n_warps) {
    const uint32_t tail = (P.K & 31) ? (1u << (P.K & 31)) - 1u : 0xFFFFFFFFu;
    const bool have = s_row[lane] >= 0;
    for (int q = warp; 4 * q < P.KW; q += n_warps) {  // KW is a multiple of 4 here
        uint4 x = make_uint4(0, 0, 0, 0);
        if (have) x = *reinterpret_cast<const uint4*>(stage + lane * a.stage_stride + 4 * q);
        if (4 * q + 4 == P.KW) x.w &= tail;
        const uint32_t t0 = warp_transpose32(x.x, lane), t1 = warp_transpose32(x.y, lane);
        const uint32_t t2 = warp_transpose32(x.z, lane), t3 = warp_transpose32(x.w, lane);
        uint32_t* dst = T + (4 * q) * 32 + lane;
        dst[0] = t0; dst[32] = t1; dst[64] = t2; dst[96] = t3;
    }
    if (warp == 0) T[P.KW * 32 + lane] = 0u;  // the padding class
}

// Allow bits of rows 8*rb .. 8*rb+7 for the 8 tokens whose class ids are packed in cv:
// byte i of (lo, hi) belongs to row 8*rb + i, bit j of it to token j of the octet.
__device__ __forceinline__ void octet_allow_bits(const uint4& cv, const uint32_t* T, int rb, bool active, uint32_t& lo,
                                                 uint32_t& hi) {
    lo = hi = 0;
    if (!active) return;
    const uint32_t w0 = T[cv.x & 0xFFFFu], w1 = T[cv.x >> 16], w2 = T[cv.y & 0xFFFFu], w3 = T[cv.y >> 16];
    const uint32_t w4 = T[cv.z & 0xFFFFu], w5 = T[cv.z >> 16], w6 = T[cv.w & 0xFFFFu], w7 = T[cv.w >> 16];
    const uint32_t sel = uint32_t(rb) | (uint32_t(4 + rb) << 4);  // byte rb of both operands
    lo = __byte_perm(__byte_perm(w0, w1, sel), __byte_perm(w2, w3, sel), 0x5410);
    hi = __byte_perm(__byte_perm(w4, w5, sel), __byte_perm(w6, w7, sel), 0x5410);
    transpose8x8(lo, hi);
}

// Lowest allowed token of a row, found from the class side: the first member of every allowed
// class (the member lists are ascending), minimum over the classes this caller looks at
// (words l, l+n, ... of the class mask). Returns (token << 32) | representative, ~0 if none.
// Only rows whose allowed logits are all -inf (or that allow nothing) come here.
__device__ __forceinline__ unsigned long long first_allowed_share(const StepArgs& a, const PartDev& P, int row, int l,
                                                                  int n) {
    unsigned long long best = ~0ull;
    const uint32_t* cm = a.class_mask + int64_t(row) * a.cm_stride;
    for (int kw = l; kw < P.KW; kw += n) {
        uint32_t w = cm[kw];
        if (kw == P.KW - 1 && (P.K & 31)) w &= (1u << (P.K & 31)) - 1u;
        while (w) {
            const int k = kw * 32 + __ffs(w) - 1;
            w &= w - 1u;
            const unsigned long long cand =
                (static_cast<unsigned long long>(P.tok[P.off[k]]) << 32) | static_cast<unsigned int>(P.r[k]);
            best = cand < best ? cand : best;
        }
    }
    return best;
}

__device__ __forceinline__ void write_row_outputs(const StepArgs& a, int row, float m, float s, unsigned long long pick) {
    int tok = -1, repv = -1;
    float lsev = -INFINITY, lpa = -INFINITY;
    if (pick != ~0ull) {
        tok = int(pick >> 32);
        repv = int(pick & 0xFFFFFFFFull);
        if (m > kRefFloor && s > 0.f) {
            const float l = logf(s);
            lsev = m + l;
            lpa = -l;
        }
    } else {
        atomicAdd(a.status + 0, 1);
    }
    a.argmax[row] = tok;
    if (a.rep) a.rep[row] = repv;
    if (a.lse) a.lse[row] = lsev;
    if (a.logp_argmax) a.logp_argmax[row] = lpa;
}

template <int DT>
__device__ __forceinline__ void warp_finalize_row(const StepArgs& a, const PartDev& P, int row, float m, float s,
                                                  int pos, int lane) {
    unsigned long long cand = ~0ull;
    if (pos == kNoPos) {
        cand = first_allowed_share(a, P, row, lane, 32);
    } else {
        // a position means that m is a finite allowed logit; the row is already masked in memory (disallowed
        // logits read -inf), so the first token of the octet that holds the value m is the choice. Its
        // representative is fetched side by side with the logit.
        // the position is the first octet of the 8 or 16 tokens its producer handled together: 16 lanes look
        const int t = 8 * pos + lane;
        if (lane < 16 && pos >= 0 && t < a.V) {
            const float z = ldcg_elem<DT>(reinterpret_cast<const char*>(a.logits) + logits_row(a, row) * a.row_stride * (DT == kBF16 ? 2 : 4), t);
            const int repv = __ldg(P.trep + t);
            bool ok = z == m;
            if (a.masks_per_row > 0) {  // the logits were left as they are: ask this row's class mask
                const int k = __ldg(P.c32 + t);
                ok = ok && ((__ldg(a.class_mask + int64_t(row) * a.cm_stride + (k >> 5)) >> (k & 31)) & 1u);
            }
            if (ok) cand = (static_cast<unsigned long long>(t) << 32) | static_cast<unsigned int>(repv);
        }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, cand, d);
        cand = other < cand ? other : cand;
    }
    if (lane == 0) write_row_outputs(a, row, m, s, cand);
}

// The octets past the last whole vector of a row (the ragged one when V is not a multiple of
// 8, and the padding octets up to the end of the last vocab-mask word): at most four per row.
// One warp takes them after the streaming loop, lane r = row slot r, token by token straight
// from the class-id vector and the row's class mask (compact code, run by one block per group).
template <int DT>
__device__ __forceinline__ Partial dense_tail_octets(const StepArgs& a, const PartDev& P, int row, int o_first, int o_end,
                                                     float scale) {
    constexpr int ES = DT == kBF16 ? 2 : 4;
    float m = -INFINITY, s = 0.f;
    int pos = kNoPos;
    if (row < 0) return Partial{m, s, pos, 0};
    const uint32_t* cm = a.class_mask + int64_t(row) * a.cm_stride;
    char* rowp = reinterpret_cast<char*>(a.logits) + logits_row(a, row) * a.row_stride * ES;
    uint8_t* vmp = a.vocab_mask ? reinterpret_cast<uint8_t*>(a.vocab_mask) + int64_t(row) * a.vm_stride * 4 : nullptr;
    for (int o = o_first; o < o_end; ++o) {
        uint32_t byte = 0;
        for (int j = 0; j < 8; ++j) {
            const int t = 8 * o + j;
            if (t >= a.V) break;
            const int k = P.c32[t];
            if ((cm[k >> 5] >> (k & 31)) & 1u) {
                byte |= 1u << j;
                const float z = load_elem<DT>(rowp, t);
                if (z > m) pos = o;
                const float ref_old = fmaxf(m, kRefFloor);
                m = fmaxf(m, z);
                const float ref = fmaxf(m, kRefFloor);
                s = fmaf(s, ex2f((ref_old - ref) * scale), ex2f((z - ref) * scale));
            } else if (a.masks_per_row == 0) {
                store_neg_inf<DT>(rowp, t);
            }
        }
        if (vmp) vmp[o] = uint8_t(byte);
    }
    return Partial{m, s, pos, 0};
}

// Where the (max, sum-exp, position) states of a row go: every warp that streamed a row batch
// publishes one state per row in its own slot, slot = split * WT + wt, and the block that owns the
// end of the vocabulary adds the state of the octets past the last whole vector in the last
// slot. a.slots = S * WT + 1 states per row, rows of a group side by side.
__device__ __forceinline__ Partial* row_slots(const StepArgs& a, int g, int row_slot) {
    return a.partials + (int64_t(g) * kGroupRows + row_slot) * a.slots;
}

// After the streaming loop of a dense block: the warp that is told to (warp 0 of the block that
// owns the end of the vocabulary) handles the tail octets, lane r = row slot r.
template <int DT>
__device__ __forceinline__ void publish_tail_octets(const StepArgs& a, const PartDev& P, int g, const int* s_row, int lane,
                                                    int tail_first, int tail_end, float scale = kLog2e) {
    const Partial p = dense_tail_octets<DT>(a, P, s_row[lane], tail_first, tail_end, scale);
    if (s_row[lane] >= 0) row_slots(a, g, lane)[a.slots - 1] = p;
}
// The same into any array of states: row slot r's state goes to base[r * stride + slot].
template <int DT>
__device__ __forceinline__ void publish_tail_octets_to(const StepArgs& a, const PartDev& P, const int* s_row, int lane,
                                                       int tail_first, int tail_end, float scale, Partial* base, int stride,
                                                       int slot) {
    const Partial p = dense_tail_octets<DT>(a, P, s_row[lane], tail_first, tail_end, scale);
    if (s_row[lane] >= 0) base[lane * stride + slot] = p;
}

// ---------------------------------------------------------------------------------------
// Second kernel of a dense step: one block per (group, row slot). Folds the row's published
// states, finds the winning token among the 8 tokens of the winning octet (8 lanes side by side,
// each fetching its candidate's representative as well) and writes the row's results.
// ---------------------------------------------------------------------------------------
constexpr int kFinalizeThreads = 256;

template <int DT>
__global__ void __launch_bounds__(kFinalizeThreads) k_finalize_rows(const __grid_constant__ StepArgs a) {
    pdl_prologue();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = blockIdx.x / kGroupRows, j = blockIdx.x - g * kGroupRows;
    if (a.n_groups && g >= __ldg(a.n_groups)) return;
    int row;
    if (a.group_rows) {
        row = a.group_rows[g * kGroupRows + j];
    } else {
        row = g * kGroupRows + j;
        if (row >= a.B) row = -1;
    }
    if (row < 0) return;
    if (a.row_mode && a.row_mode[row]) return;  // automatic mode: the class-list kernel has finished this row
    const PartDev P = a.group_part ? a.parts[a.group_part[g]] : a.p0;
    const Partial* src = row_slots(a, g, j);
    // Two passes over the states, which stay in registers (up to four per thread, all loads in flight together):
    // first the row maximum (shuffles and max only), then every state's sum brought to that maximum with one
    // exponential per state, summed, and the lowest position among the states that hold the maximum. No
    // exponential sits inside a reduction chain, and the three reductions run side by side.
    constexpr int kWarps = kFinalizeThreads / 32;
    __shared__ float s_max[kWarps], s_sum[kWarps];
    __shared__ int s_pos[kWarps];
    auto fetch = [&](int base, int4 (&v)[4]) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int sp = base + u * kFinalizeThreads + tid;
            v[u] = make_int4(__float_as_int(-INFINITY), 0, kNoPos, 0);
            if (sp < a.slots) v[u] = __ldcg(reinterpret_cast<const int4*>(src + sp));
        }
    };
    int4 v0[4];
    fetch(0, v0);
    float M = fmaxf(fmaxf(__int_as_float(v0[0].x), __int_as_float(v0[1].x)), fmaxf(__int_as_float(v0[2].x), __int_as_float(v0[3].x)));
    for (int base = 4 * kFinalizeThreads; base < a.slots; base += 4 * kFinalizeThreads) {  // more than 1024 states: rare
        int4 w[4];
        fetch(base, w);
        M = fmaxf(M, fmaxf(fmaxf(__int_as_float(w[0].x), __int_as_float(w[1].x)), fmaxf(__int_as_float(w[2].x), __int_as_float(w[3].x))));
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, d));
    if (lane == 0) s_max[warp] = M;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, s_max[w]);
    const float Mf = fmaxf(M, kRefFloor);
    float sum = 0.f;
    int pos = kNoPos;
    auto gather = [&](const int4 (&v)[4]) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float m = __int_as_float(v[u].x);
            sum = fmaf(__int_as_float(v[u].y), ex2f((fmaxf(m, kRefFloor) - Mf) * kLog2e), sum);
            pos = (m == M) ? min(pos, v[u].z) : pos;
        }
    };
    gather(v0);
    for (int base = 4 * kFinalizeThreads; base < a.slots; base += 4 * kFinalizeThreads) {
        int4 w[4];
        fetch(base, w);
        gather(w);
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        sum += __shfl_xor_sync(0xFFFFFFFFu, sum, d);
        pos = min(pos, __shfl_xor_sync(0xFFFFFFFFu, pos, d));
    }
    if (lane == 0) {
        s_sum[warp] = sum;
        s_pos[warp] = pos;
    }
    __syncthreads();
    if (warp != 0) return;
    sum = 0.f;
    pos = kNoPos;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {  // every lane of warp 0 takes the same eight values in the same order
        sum += s_sum[w];
        pos = min(pos, s_pos[w]);
    }
    warp_finalize_row<DT>(a, P, row, M, sum, pos, lane);
}

// The same for rows with few published states (at most 4 per lane: large batches, where a group is
// shared by few blocks): one warp per row, 8 rows per block, no block-level step at all.
constexpr int kFinalizeWarpStates = 128;

template <int DT>
__global__ void __launch_bounds__(256) k_finalize_rows_warp(const __grid_constant__ StepArgs a) {
    pdl_prologue();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int idx = blockIdx.x * 8 + warp;  // (group, row slot)
    const int g = idx / kGroupRows, j = idx - g * kGroupRows;
    if (a.n_groups && g >= __ldg(a.n_groups)) return;
    int row;
    if (a.group_rows) {
        row = a.group_rows[g * kGroupRows + j];
    } else {
        row = g * kGroupRows + j;
        if (row >= a.B) row = -1;
    }
    if (row < 0) return;
    if (a.row_mode && a.row_mode[row]) return;  // automatic mode: the class-list kernel has finished this row
    const PartDev P = a.group_part ? a.parts[a.group_part[g]] : a.p0;
    const Partial* src = row_slots(a, g, j);
    int4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int sp = u * 32 + lane;
        v[u] = make_int4(__float_as_int(-INFINITY), 0, kNoPos, 0);
        if (sp < a.slots) v[u] = __ldcg(reinterpret_cast<const int4*>(src + sp));
    }
    float m0 = __int_as_float(v[0].x), s0 = __int_as_float(v[0].y), m1 = __int_as_float(v[1].x), s1 = __int_as_float(v[1].y);
    int p0 = v[0].z, p1 = v[1].z;
    partial_merge(m0, s0, p0, __int_as_float(v[2].x), __int_as_float(v[2].y), v[2].z);
    partial_merge(m1, s1, p1, __int_as_float(v[3].x), __int_as_float(v[3].y), v[3].z);
    partial_merge(m0, s0, p0, m1, s1, p1);
    partial_warp_allreduce(m0, s0, p0);
    warp_finalize_row<DT>(a, P, row, m0, s0, p0, lane);
}

// One whole-vector octet of one row: mask, write back, note the vocab-mask byte, fold into the
// row state.
template <int DT>
__device__ __forceinline__ void dense_octet_row(Octet<DT>& oc, char* rowp, uint8_t* vmp, int o, uint32_t byte,
                                                RowAcc& acc, bool wide, bool write_back = true) {
    float f[8];
    oc.mask(byte, f);
    if (write_back) oc.store(rowp, o, wide);
    if (vmp) vmp[o] = uint8_t(byte);
    acc.add_octet(f, o);
}

// Order-preserving map between floats and signed integers (for the integer warp reductions).
__device__ __forceinline__ int float_order_key(float x) {
    const int i = __float_as_int(x);
    return i >= 0 ? i : i ^ 0x7FFFFFFF;
}
__device__ __forceinline__ float float_from_order_key(int k) { return __int_as_float(k >= 0 ? k : k ^ 0x7FFFFFFF); }

// Reduce the 8 row states of a warp over its 32 lanes and publish them in the warp's slot of each row.
// The state of row slot r goes to base[r * stride + slot] (global scratch, or the block's shared array).
__device__ __forceinline__ void warp_rows_publish_to(RowAcc (&acc)[kBatchRows], int live, int rb, int lane, float scale,
                                                     Partial* base, int stride, int slot) {
    // Two passes, no exponential inside a reduction chain: the maximum of every row over the lanes (one integer
    // warp reduction each), every lane's sum brought to it with one exponential, the lowest position among the
    // lanes that hold the maximum (one more integer reduction), and the eight sums reduced by recursive halving
    // (lanes trade half of their rows with the lane 16 away, then 2 of 4 with the lane 8 away, then 1 of 2; two
    // butterfly steps finish the single row left).
    float M[kBatchRows], w[kBatchRows];
    int pos[kBatchRows];
#pragma unroll
    for (int i = 0; i < kBatchRows; ++i) M[i] = float_from_order_key(__reduce_max_sync(0xFFFFFFFFu, float_order_key(acc[i].m)));
#pragma unroll
    for (int i = 0; i < kBatchRows; ++i) {
        w[i] = M[i] > kRefFloor ? acc[i].s * ex2f(-fmaf(M[i], scale, acc[i].nrl)) : 0.f;
        pos[i] = __reduce_min_sync(0xFFFFFFFFu, acc[i].m == M[i] ? acc[i].pos : kNoPos);
    }
#pragma unroll
    for (int half = 4; half >= 1; half >>= 1) {
        const int d = 4 * half;  // 16, 8, 4
        const bool up = lane & d;
#pragma unroll
        for (int k = 0; k < half; ++k) {
            const float keep = up ? w[k + half] : w[k];
            const float send = up ? w[k] : w[k + half];
            w[k] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, d);
        }
    }
    w[0] += __shfl_xor_sync(0xFFFFFFFFu, w[0], 2);
    w[0] += __shfl_xor_sync(0xFFFFFFFFu, w[0], 1);
    const int i = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);  // the row this lane ended with
    float Mi = M[0];
    int pi = pos[0];
#pragma unroll
    for (int k = 1; k < kBatchRows; ++k) {
        Mi = i == k ? M[k] : Mi;
        pi = i == k ? pos[k] : pi;
    }
    if ((lane & 3) == 0 && i < live) base[(rb * kBatchRows + i) * stride + slot] = Partial{Mi, w[0], pi, 0};
}
__device__ __forceinline__ void warp_rows_publish(const StepArgs& a, RowAcc (&acc)[kBatchRows], int live, int g, int slot,
                                                  int rb, int lane, float scale = kLog2e) {
    warp_rows_publish_to(acc, live, rb, lane, scale, row_slots(a, g, 0), a.slots, slot);
}

// Fold up to `n` states (16 bytes each, read through L2) with the lanes of a warp side by side; every lane returns
// the merged state. Four loads per lane are in flight together.
__device__ __forceinline__ void warp_fold_states(const Partial* src, int n, int lane, float& m, float& s, int& pos) {
    m = -INFINITY;
    s = 0.f;
    pos = kNoPos;
    for (int base = 0; base < n; base += 128) {
        int4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int sp = base + u * 32 + lane;
            v[u] = make_int4(__float_as_int(-INFINITY), 0, kNoPos, 0);
            if (sp < n) v[u] = __ldcg(reinterpret_cast<const int4*>(src + sp));
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) partial_merge(m, s, pos, __int_as_float(v[u].x), __int_as_float(v[u].y), v[u].z);
    }
    partial_warp_allreduce(m, s, pos);
}

// ---------------------------------------------------------------------------------------
// Fused dense step, register version: expand + mask in place + (max, sum-exp, position) per
// row, logits fetched with 16-byte loads straight into registers (rows 16-byte aligned).
// Grid: n_groups * S thread blocks; block (g, split) owns octets [split*per_split, ...) of the
// 32 rows of group g. Warps are arranged WT (along tokens) x WR (row batches of 8).
// ---------------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(256) k_step_dense(const __grid_constant__ StepArgs a) {
    extern __shared__ __align__(128) uint32_t smem[];
    uint32_t* T = smem;
    int* s_row = reinterpret_cast<int*>(T + a.table_words);
    uint32_t* stage = reinterpret_cast<uint32_t*>(s_row + kGroupRows);

    pdl_prologue();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, n_warps = blockDim.x >> 5;
    const int g = blockIdx.x / a.S, split = blockIdx.x - g * a.S;
    if (a.n_groups && g >= __ldg(a.n_groups)) return;
    const int part = group_rows_setup(a, g, s_row, tid);
    __syncthreads();
    const PartDev P = a.group_part ? a.parts[part] : a.p0;
    const int nrow = __popc(__ballot_sync(0xFFFFFFFFu, s_row[lane] >= 0));
    if (a.stage_stride) {
        stage_class_masks(a, P, s_row, stage, warp, lane, n_warps);
        __syncthreads();
    }
    build_class_table(a, P, s_row, T, stage, warp, lane, n_warps);
    __syncthreads();

    const int wt = warp % a.WT, wr = warp / a.WT, WR = n_warps / a.WT;
    const int n_octets = 4 * a.VW, n_full = a.V >> 3;
    const int o_begin = split * a.per_split;
    const int o_end = min(o_begin + a.per_split, n_octets);
    const int o_vec_end = min(o_end, n_full);
    constexpr int ES = DT == kBF16 ? 2 : 4;
    uint8_t* vm8 = reinterpret_cast<uint8_t*>(a.vocab_mask);

    for (int rb = wr; rb * kBatchRows < nrow; rb += WR) {
        RowAcc acc[kBatchRows];
        char* rowp[kBatchRows];
        uint8_t* vmp[kBatchRows];
#pragma unroll
        for (int i = 0; i < kBatchRows; ++i) {
            acc[i].init();
            const int row = s_row[min(rb * kBatchRows + i, kGroupRows - 1)];
            rowp[i] = reinterpret_cast<char*>(a.logits) + logits_row(a, max(row, 0)) * a.row_stride * ES;
            vmp[i] = vm8 ? vm8 + int64_t(max(row, 0)) * a.vm_stride * 4 : nullptr;
        }
        const int live = min(kBatchRows, nrow - rb * kBatchRows);

        for (int o0 = o_begin + wt * 32; o0 < o_vec_end; o0 += a.WT * 32) {
            const int o = o0 + lane;
            const bool active = o < o_vec_end;
            Octet<DT> oc[kBatchRows];
#pragma unroll
            for (int i = 0; i < kBatchRows; ++i)
                if (i < live && active) oc[i].load(rowp[i], o);
            uint32_t lo, hi;
            uint4 cv = make_uint4(0, 0, 0, 0);
            if (active) cv = __ldg(reinterpret_cast<const uint4*>(P.c16) + o);
            octet_allow_bits(cv, T, rb, active, lo, hi);
#pragma unroll
            for (int i = 0; i < kBatchRows; ++i) {
                if (i < live && active) {
                    const uint32_t byte = ((i < 4 ? lo : hi) >> (8 * (i & 3))) & 0xFFu;
                    dense_octet_row<DT>(oc[i], rowp[i], vmp[i], o, byte, acc[i], a.wide != 0, a.masks_per_row == 0);
                }
            }
        }
        warp_rows_publish(a, acc, live, g, split * a.WT + wt, rb, lane);
    }
    // the block that reaches the end of the vocabulary takes the octets past the last whole vector
    if (warp == 0 && o_end == n_octets) publish_tail_octets<DT>(a, P, g, s_row, lane, max(o_begin, n_full), o_end);
}

// ---------------------------------------------------------------------------------------
// Fused dense step, pipelined version. Same decomposition as above, but the logits reach the
// SM through bulk asynchronous copies: every warp runs its own ring of `depth` stages in
// shared memory, each stage holding 32 octets of 8 rows plus the 32 octets of class ids,
// filled by copies that lane 0 issues `depth` work items ahead and that signal an mbarrier.
// The first copies are started before the class table is built. The lanes read their 16
// bytes per row from shared memory, so no registers wait on memory and the copies of later
// items overlap the arithmetic of this one. Masked logits go back with 16-byte stores.
// ---------------------------------------------------------------------------------------
// OPL: octets a lane handles per row of an item (1, or 2 for bf16: 32 bytes per lane and row either way for OPL = 2
// and for f32). A chunk is the 32 * OPL octets the lanes of a warp cover together.
template <int DT, int OPL>
struct PipeGeom {
    static constexpr int kOctetBytes = DT == kBF16 ? 16 : 32;
    static constexpr int kBoxBytes = kBatchRows * 32 * kOctetBytes;        // one tiled copy: 8 rows of 32 octets
    static constexpr int kRowBytes = 32 * OPL * kOctetBytes;               // one row of a stage
    static constexpr int kChunkOctets = 32 * OPL;
    static constexpr int kStageBytes = kBatchRows * kRowBytes + kChunkOctets * 16;  // + class ids of the chunk
};

// Where the rows of a batch live. With consecutive rows (CONSEC) the address of row i is one
// wide multiply-add from the batch's base; otherwise each row has its own base pointer.
struct BatchAddr {
    char* item_base;      // CONSEC: logits of row 0 of the batch at this lane's octet
    uint8_t* vm_item;     // CONSEC: vocab-mask byte of row 0 at this lane's octet (or null)
    uint32_t row_bytes;   // CONSEC: bytes between rows of the logits
    uint32_t vm_bytes;    // CONSEC: bytes between rows of the vocab mask
};

// One work item of a warp: the 32 * OPL octets of a chunk for the 8 rows of a batch, read from the stage `src`;
// this lane's OPL octets of row i lie at src + i * srow + lane_off. n_act: how many of the lane's octets are whole
// vectors of the row (OPL everywhere except at the end of the vocabulary).
// FULL: all 8 rows live and every lane's octets inside the whole-vector range (no per-row tests).
template <int DT, int OPL, bool FULL, bool CONSEC>
__device__ __forceinline__ void pipe_consume_item(const char* src, uint32_t lane_off, uint32_t srow, const uint32_t* T, int rb,
                                                  int live, int n_act, int o, int lane, const BatchAddr& ba,
                                                  char* const (&rowp)[kBatchRows], uint8_t* const (&vmp)[kBatchRows],
                                                  RowAcc (&acc)[kBatchRows], float scale, bool wide) {
    using G = PipeGeom<DT, OPL>;
    uint32_t lo[OPL], hi[OPL];
#pragma unroll
    for (int q = 0; q < OPL; ++q) {
        const bool act = FULL || q < n_act;
        uint4 cv = make_uint4(0, 0, 0, 0);
        if (act) cv = *reinterpret_cast<const uint4*>(src + kBatchRows * G::kRowBytes + (lane * OPL + q) * 16);
        octet_allow_bits(cv, T, rb, act, lo[q], hi[q]);
    }
    const bool both = FULL || n_act == OPL;
#pragma unroll
    for (int i = 0; i < kBatchRows; ++i) {
        if (FULL || (i < live && n_act > 0)) {
            Octet<DT> oc[OPL];
            float f[8 * OPL];
            uint32_t bytes = 0;
#pragma unroll
            for (int q = 0; q < OPL; ++q) {
                const uint32_t byte = ((i < 4 ? lo[q] : hi[q]) >> (8 * (i & 3))) & 0xFFu;  // 0 for an octet past the range
                if (FULL || q < n_act)
                    oc[q].load_shared_at(src + i * srow + lane_off + q * G::kOctetBytes);
                else
                    oc[q].fill_neg_inf();
                oc[q].mask(byte, f + 8 * q);
                bytes |= byte << (8 * q);
            }
            char* zp = CONSEC ? ptr_mad(ba.item_base, i, ba.row_bytes) : rowp[i] + size_t(o) * G::kOctetBytes;
            char* vp = CONSEC ? (ba.vm_item ? ptr_mad(reinterpret_cast<char*>(ba.vm_item), i, ba.vm_bytes) : nullptr)
                              : (vmp[i] ? reinterpret_cast<char*>(vmp[i]) + o : nullptr);
            if (OPL == 1) {
                oc[0].store_at(zp, wide);
                if (vp) st_global_u8(vp, bytes);
            } else {
                if (both && wide) {
                    st_stream32(zp, oc[0].raw(), oc[OPL - 1].raw());
                } else {
                    oc[0].store_at(zp);
                    if (both) oc[OPL - 1].store_at(zp + G::kOctetBytes);
                }
                if (vp) {
                    if (both) st_global_u16(vp, bytes); else st_global_u8(vp, bytes & 0xFFu);
                }
            }
            acc[i].template add_values<8 * OPL>(f, o, scale);
        }
    }
}

// TMAP: the 8 rows of a batch are consecutive rows of the logits matrix and arrive as tiled 2-D copies
// through `tmap` (box = 256 elements x 8 rows: one per chunk, two for a chunk of 512 bf16 tokens);
// otherwise one bulk copy per row. OPL: octets per lane and row (see PipeGeom).
// LBT / MINB: launch bounds (threads per block, blocks per SM) the variant is compiled for; they set
// the register budget: (512, 1) 128 registers, (384, 1) 168, (320, 2) 96, (256, 3) 80. TEMPERED: the sums
// are of exp(z / T) with the step's temperature (sampling steps); otherwise T = 1 is compiled in.
template <int DT, int OPL, bool TMAP, int LBT, int MINB, bool TEMPERED>
__global__ void __launch_bounds__(LBT, MINB) k_step_dense_pipe(const __grid_constant__ StepArgs a,
                                                         const __grid_constant__ CUtensorMap tmap) {
    using G = PipeGeom<DT, OPL>;
    extern __shared__ __align__(128) uint32_t smem[];
    uint32_t* T = smem;
    int* s_row = reinterpret_cast<int*>(T + a.table_words);
    const int n_warps = blockDim.x >> 5;
    uint64_t* bars = reinterpret_cast<uint64_t*>(s_row + kGroupRows);  // n_warps * depth
    int* ring_info = reinterpret_cast<int*>(bars + n_warps * a.depth);         // n_warps * depth
    char* ring = reinterpret_cast<char*>(bars) + ((n_warps * a.depth * 12 + 127) & ~127);  // keeps 128-byte alignment
    // The staging area of the class masks is dead once the table is built. Where shared memory is short it
    // shares the space of the first warps' rings; those warps then start their copies after the table.
    uint32_t* stage = a.stage_alias ? reinterpret_cast<uint32_t*>(ring)
                                    : reinterpret_cast<uint32_t*>(ring + size_t(n_warps) * a.depth * G::kStageBytes);
    __shared__ uint64_t cm_bar;

    // Without a row plan nothing of the set-up reads memory (the rows of the group are g*32 .. g*32+31, its
    // partition is part0): it runs while the kernel in front is still finishing, and the wait for that kernel
    // comes just before the first copies. With a row plan the wait comes first, as the plan is read at once.
    pdl_launch_dependents();
    const bool implicit = !a.group_rows;
    if (!implicit) pdl_wait();
    const float scale = TEMPERED ? a.scale : kLog2e;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = blockIdx.x / a.S, split = blockIdx.x - g * a.S;
    if (a.n_groups && g >= __ldg(a.n_groups)) return;
    const bool early_cm = a.cm_bulk && implicit;
    if (early_cm && tid == 0) {
        mbar_init(&cm_bar, 1);
        mbar_init_fence();
        mbar_expect_tx(&cm_bar, uint32_t(min(kGroupRows, a.B - g * kGroupRows)) * uint32_t(a.p0.KW) * 4u);
        if (TMAP) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");
    }
    const int part = group_rows_setup(a, g, s_row, tid);
    __syncthreads();
    const PartDev P = a.group_part ? a.parts[part] : a.p0;
    const int nrow = __popc(__ballot_sync(0xFFFFFFFFu, s_row[lane] >= 0));

    const int depth = a.depth;
    const int wt = warp % a.WT, wr = warp / a.WT, WR = n_warps / a.WT;
    const int n_octets = 4 * a.VW, n_full = a.V >> 3;
    constexpr int ES = DT == kBF16 ? 2 : 4;
    uint8_t* vm8 = reinterpret_cast<uint8_t*>(a.vocab_mask);
    char* my_ring = ring + size_t(warp) * depth * G::kStageBytes;
    uint64_t* bar = bars + warp * depth;

    // Work items: (row batch, chunk of 32 whole-vector octets). A warp owns the row batches rb = wr,
    // wr+WR, ...; the chunks of a row batch are dealt round-robin to the warps of the group that own it
    // (warp index among them, then a stride of their number), so that at any moment the group's blocks
    // read neighbouring pieces of the same rows: measured 5 % faster on long steps than one contiguous
    // range per block, and as fast as handing chunks out through global counters.
    // In a sampling step (TEMPERED) the states of a row must follow the token order: every warp slot then
    // takes one contiguous run of run_chunks chunks instead.
    // The number of chunks is rarely a multiple of the number of warp slots, so some slots get one chunk more than
    // the others; the deal starts at a different slot for every row batch (rot_chunks further on), which spreads the
    // extra chunks evenly over the warps and the blocks instead of giving the first ones one more in every row batch.
    const int n_chunks = (n_full + G::kChunkOctets - 1) / G::kChunkOctets;
    const int stride_chunks = TEMPERED ? 1 : a.S * a.WT;  // round-robin: warps that share a row batch of the group
    auto first_chunk_of = [&](int rb) {  // this warp's first chunk of row batch rb
        if (TEMPERED) return (split * a.WT + wt) * a.run_chunks;
        int c = split * a.WT + wt - rb * a.rot_chunks;
        c %= stride_chunks;
        return c < 0 ? c + stride_chunks : c;
    };
    const int chunk_end = TEMPERED ? min(first_chunk_of(0) + a.run_chunks, n_chunks) : n_chunks;
    int* const slot_info = ring_info + warp * depth; // (rb << 24) | chunk of the item in each slot, -1 = no more items

    // automatic mode: bit r = row slot r was finished by the class-list kernel (set after the wait below)
    uint32_t rows_done = 0u;
    auto batch_done = [&](int rb) {
        const int n = min(kBatchRows, nrow - rb * kBatchRows);
        const uint32_t all = n >= 8 ? 0xFFu : (1u << n) - 1u;
        return ((rows_done >> (rb * kBatchRows)) & 0xFFu) == all;
    };
    // producer cursor (meaningful in lane 0)
    int p_rb = wr, p_slot = 0, p_issued = 0, p_chunk = 0;
    bool p_first = true, p_done = wr * kBatchRows >= nrow, p_end = false;
    auto issue_next = [&]() {
        int chunk = -1;
        while (!p_done) {
            if (p_first && rows_done && batch_done(p_rb)) {  // nothing left to do for this row batch
                p_rb += WR;
                p_done = p_rb * kBatchRows >= nrow;
                continue;
            }
            if (p_first) {
                chunk = first_chunk_of(p_rb);
                p_first = false;
            } else {
                chunk = p_chunk + stride_chunks;
            }
            p_chunk = chunk;
            if (chunk < chunk_end) break;
            chunk = -1;  // this row batch is handed out completely: on to the warp's next one
            p_rb += WR;
            p_first = true;
            p_done = p_rb * kBatchRows >= nrow;
        }
        if (chunk < 0) {
            slot_info[p_slot] = -1;
            p_end = true;
            return;
        }
        slot_info[p_slot] = (p_rb << 24) | chunk;
        const int o0 = chunk * G::kChunkOctets;
        char* dst = my_ring + size_t(p_slot) * G::kStageBytes;
        const uint32_t nvec = uint32_t(min(n_full - o0, G::kChunkOctets));  // >= 1: chunk < n_chunks
        if (TMAP) {
            // a box holds 32 octets of the 8 rows; the second box of a two-octet chunk is fetched only if the chunk
            // reaches into it (its lanes are idle otherwise); parts of a box past V or past the last row are filled in
            const int nbox = (OPL == 2 && nvec > 32u) ? 2 : 1;
            mbar_expect_tx(bar + p_slot, uint32_t(nbox * G::kBoxBytes) + nvec * 16u);
            tma_g2s_2d(dst, &tmap, o0 * 8, s_row[p_rb * kBatchRows], bar + p_slot);
            if (nbox == 2) tma_g2s_2d(dst + G::kBoxBytes, &tmap, o0 * 8 + 256, s_row[p_rb * kBatchRows], bar + p_slot);
        } else {
            const int live = min(kBatchRows, nrow - p_rb * kBatchRows);
            const uint32_t row_bytes = nvec * G::kOctetBytes;
            mbar_expect_tx(bar + p_slot, uint32_t(live) * row_bytes + nvec * 16u);
            for (int i = 0; i < live; ++i) {
                const int row = s_row[p_rb * kBatchRows + i];
                bulk_g2s(dst + i * G::kRowBytes,
                         reinterpret_cast<const char*>(a.logits) + (int64_t(row) * a.row_stride * ES + int64_t(o0) * 8 * ES),
                         row_bytes, bar + p_slot);
            }
        }
        bulk_g2s(dst + kBatchRows * G::kRowBytes, reinterpret_cast<const char*>(P.c16) + size_t(o0) * 16, nvec * 16u, bar + p_slot);
        ++p_issued;
        if (++p_slot == depth) p_slot = 0;
    };

    if (lane == 0) {
        for (int d = 0; d < depth; ++d) mbar_init(bar + d, 1);
        if (warp == 0 && !early_cm) mbar_init(&cm_bar, 1);
        mbar_init_fence();
    }
    if (implicit && a.prefetch_items > 0 && lane == 0 && !p_done) {
        // While the kernel in front is finishing, DRAM has little to do: ask this warp's first work items (and the
        // group's class masks) into the L2. These are hints only: they deliver nothing, and whatever the kernel in
        // front may still write reaches the same L2, so nothing stale can be read after the wait.
        const int row0 = g * kGroupRows + wr * kBatchRows;
        const int live0 = min(kBatchRows, nrow - wr * kBatchRows);
        int chunk = first_chunk_of(wr);
        for (int d = 0; d < a.prefetch_items && chunk < chunk_end; ++d, chunk += TEMPERED ? 1 : stride_chunks) {
            const int o0 = chunk * G::kChunkOctets;
            const uint32_t nvec = uint32_t(min(n_full - o0, G::kChunkOctets));
            if (TMAP) {
                tma_prefetch_2d(&tmap, o0 * 8, row0);
                if (OPL == 2 && nvec > 32u) tma_prefetch_2d(&tmap, o0 * 8 + 256, row0);
            } else {
                for (int i = 0; i < live0; ++i)
                    bulk_prefetch(reinterpret_cast<const char*>(a.logits) + (int64_t(row0 + i) * a.row_stride * ES + int64_t(o0) * 8 * ES),
                                  nvec * G::kOctetBytes);
            }
        }
        if (warp == 0 && a.cm_bulk)
            for (int r = 0; r < nrow; ++r)
                bulk_prefetch(a.class_mask + int64_t(g * kGroupRows + r) * a.cm_stride, uint32_t(a.p0.KW) * 4u);
    }
    if (implicit) pdl_wait();
    // automatic mode: row batches that allow few tokens were finished by the class-list kernel in front and get no
    // work items here (that kernel decides for the 8 row slots of a batch together).
    if (a.row_mode) {
        rows_done = __ballot_sync(0xFFFFFFFFu, s_row[lane] >= 0 && a.row_mode[s_row[lane]] != 0);
        if (rows_done == __ballot_sync(0xFFFFFFFFu, s_row[lane] >= 0)) return;  // the whole group is done
    }
    if (early_cm) {
        // the class masks first (everything waits for them): the rows dealt over the warps, so that no warp
        // issues more than a few copies; the barrier was set up by thread 0 before the block met above
        const int r = warp + n_warps * lane;
        if (r < kGroupRows && g * kGroupRows + r < a.B)
            bulk_g2s(stage + r * a.stage_stride, a.class_mask + int64_t(g * kGroupRows + r) * a.cm_stride, uint32_t(a.p0.KW) * 4u,
                     &cm_bar);
    }
    if (a.cm_bulk && !early_cm) {
        __syncthreads();  // the class-mask barrier is initialised for everybody
        if (warp == 0) {
            // one bulk copy per row of the group, issued side by side by the lanes of one warp
            if (lane == 0) mbar_expect_tx(&cm_bar, uint32_t(nrow) * uint32_t(P.KW) * 4u);
            __syncwarp();
            const int row = s_row[lane];
            if (row >= 0)
                bulk_g2s(stage + lane * a.stage_stride, a.class_mask + int64_t(row) * a.cm_stride, uint32_t(P.KW) * 4u, &cm_bar);
        }
    }
    if (lane == 0 && warp >= a.hold_warps)  // hold_warps is 0 unless the staging area lies over the rings
        for (int d = 0; d < depth && !p_end; ++d) issue_next();  // in flight while the table is built
    bool failed = false;
    if (a.cm_bulk) {
        if (!mbar_wait(&cm_bar, 0)) failed = true;
        build_class_table_quads(a, P, s_row, T, stage, warp, lane, n_warps);
    } else {
        if (a.stage_stride) {
            stage_class_masks(a, P, s_row, stage, warp, lane, n_warps);
            __syncthreads();
        }
        build_class_table(a, P, s_row, T, stage, warp, lane, n_warps);
    }
    __syncthreads();
    if (__any_sync(0xFFFFFFFFu, failed) && lane == 0) atomicAdd(a.status + 3, 1);  // class masks never arrived
    failed = false;
    if (lane == 0 && warp < a.hold_warps) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the staging area was read and written by plain accesses
        for (int d = 0; d < depth && !p_end; ++d) issue_next();
    }

    int slot = 0;
    uint32_t phase = 0;
    int consumed = 0;
    // Where this warp's row states go: its own slot of the global scratch, or (fold with block-level merge) the
    // block's shared array of (row slot, warp along tokens) states
    const bool fold = !TEMPERED && a.fold != 0;
    Partial* const s_state = (!TEMPERED && a.fold_off) ? reinterpret_cast<Partial*>(reinterpret_cast<char*>(smem) + a.fold_off) : nullptr;
    Partial* const pub_base = s_state ? s_state : row_slots(a, g, 0);
    const int pub_stride = s_state ? a.WT + 1 : a.slots;
    const int my_slot = s_state ? wt : split * a.WT + wt;
    // where this lane's octets of a row sit inside a stage: two tiled copies leave two boxes of 8 rows x 32 octets
    // behind one another, anything else whole rows of the chunk
    const uint32_t lane_off = (TMAP && OPL == 2) ? uint32_t(lane >> 4) * G::kBoxBytes + uint32_t(lane & 15) * 2u * G::kOctetBytes
                                                 : uint32_t(lane) * OPL * G::kOctetBytes;
    const uint32_t srow = (TMAP && OPL == 2) ? 32u * G::kOctetBytes : uint32_t(G::kRowBytes);
    BatchAddr ba;
    ba.row_bytes = uint32_t(a.row_stride * ES);
    ba.vm_bytes = uint32_t(a.vm_stride * 4);
    RowAcc acc[kBatchRows];
    char* rowp[kBatchRows];
    uint8_t* vmp[kBatchRows];
    char* base0 = nullptr;
    uint8_t* vm0 = nullptr;
    int live = 0;
    auto open_batch = [&](int rb) {  // fresh row states and row addresses for row batch rb
#pragma unroll
        for (int i = 0; i < kBatchRows; ++i) {
            acc[i].init();
            rowp[i] = nullptr;
            vmp[i] = nullptr;
            if (!TMAP) {
                const int row = s_row[min(rb * kBatchRows + i, kGroupRows - 1)];
                rowp[i] = reinterpret_cast<char*>(a.logits) + int64_t(max(row, 0)) * a.row_stride * ES;
                vmp[i] = vm8 ? vm8 + int64_t(max(row, 0)) * a.vm_stride * 4 : nullptr;
            }
        }
        live = min(kBatchRows, nrow - rb * kBatchRows);
        const int row0 = max(s_row[min(rb * kBatchRows, kGroupRows - 1)], 0);
        base0 = reinterpret_cast<char*>(a.logits) + int64_t(row0) * a.row_stride * ES;
        vm0 = vm8 ? vm8 + int64_t(row0) * a.vm_stride * 4 : nullptr;
    };
    int cur_rb = wr;
    if (cur_rb * kBatchRows < nrow) open_batch(cur_rb);
    __syncwarp();  // slot_info written by lane 0 above
    while (cur_rb * kBatchRows < nrow) {
        const int info = slot_info[slot];
        if (info < 0) break;
        const int rb = info >> 24, o0 = (info & 0xFFFFFF) * G::kChunkOctets;
        while (cur_rb < rb) {  // the previous row batch of this warp is complete (possibly without any chunk)
            warp_rows_publish_to(acc, live, cur_rb, lane, scale, pub_base, pub_stride, my_slot);
            cur_rb += WR;
            open_batch(cur_rb);
        }
        // (the test hook lets the wait complete and then reports it as run out, so that the error path below, drain
        // loop included, runs with every copy landed)
        const bool arrived = mbar_wait(bar + slot, phase) && !a.expire_test;
        if (!__all_sync(0xFFFFFFFFu, arrived)) {
            failed = true;
            break;
        }
        const char* src = my_ring + size_t(slot) * G::kStageBytes;
        const int o = o0 + lane * OPL;
        ba.item_base = base0 + size_t(o) * G::kOctetBytes;
        ba.vm_item = vm0 ? vm0 + o : nullptr;
        if (live == kBatchRows && o0 + G::kChunkOctets <= n_full)
            pipe_consume_item<DT, OPL, true, TMAP>(src, lane_off, srow, T, rb, live, OPL, o, lane, ba, rowp, vmp, acc, scale,
                                                   a.wide != 0);
        else
            pipe_consume_item<DT, OPL, false, TMAP>(src, lane_off, srow, T, rb, live, max(0, min(OPL, n_full - o)), o, lane, ba,
                                                    rowp, vmp, acc, scale, a.wide != 0);
        ++consumed;
        if (++slot == depth) { slot = 0; phase ^= 1u; }
        __syncwarp();  // every lane has its data out of the slot before it is refilled
        if (lane == 0 && !p_end) issue_next();
        __syncwarp();  // slot_info of the refilled slot is visible to the whole warp
    }
    if (!failed) {
        // whatever row batches of this warp are left (all of them if it never got a chunk) are published too
        for (; cur_rb * kBatchRows < nrow; cur_rb += WR) {
            warp_rows_publish_to(acc, live, cur_rb, lane, scale, pub_base, pub_stride, my_slot);
            if ((cur_rb + WR) * kBatchRows < nrow) open_batch(cur_rb + WR);
        }
    } else if (lane == 0) {
        // a copy never arrived: flag it, give the copies still in flight the same bounded time to land
        // (they target this block's shared memory), and let the block leave without results
        atomicAdd(a.status + 3, 1);
        for (int k = consumed; k < p_issued; ++k) {
            mbar_wait(bar + slot, phase);
            if (++slot == depth) { slot = 0; phase ^= 1u; }
        }
    }
    // the block that reaches the end of the vocabulary takes the octets past the last whole vector
    if (warp == 0 && split == 0)
        publish_tail_octets_to<DT>(a, P, s_row, lane, n_full, n_octets, scale, pub_base, pub_stride, s_state ? a.WT : a.slots - 1);
    if (!fold && !s_state) return;
    __shared__ int s_last;
    if (s_state) {
        // first the block's own states: one per row and block goes out instead of one per row and warp
        __syncthreads();
        for (int j = warp; j < nrow; j += n_warps) {
            const int n_mine = a.WT + (split == 0 ? 1 : 0);  // only the block that owns the end of the vocabulary has a tail state
            float m = -INFINITY, s = 0.f;
            int pos = kNoPos;
            if (lane < n_mine) {
                const Partial p = s_state[j * (a.WT + 1) + lane];
                m = p.m; s = p.s; pos = p.pos;
            }
            partial_warp_allreduce(m, s, pos);
            if (lane == 0) row_slots(a, g, j)[split] = Partial{m, s, pos, 0};
        }
    }
    if (!fold) return;
    // ---- One launch per step: the group's blocks count themselves off, and the last one to finish folds the states
    // of the group's rows and writes their results (what k_finalize_rows does in a launch of its own otherwise).
    __threadfence();  // this block's states and masked logits are visible device-wide before its ticket is drawn
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(a.tickets + g, 1u) == unsigned(a.S - 1));
    __syncthreads();
    if (!s_last) return;
    __threadfence();  // the other blocks' states and masked logits, published before their tickets
    for (int j = warp; j < nrow; j += n_warps) {
        float m, s;
        int pos;
        warp_fold_states(row_slots(a, g, j), a.slots, lane, m, s, pos);
        warp_finalize_row<DT>(a, P, s_row[j], m, s, pos, lane);
    }
    if (tid == 0) a.tickets[g] = 0u;  // ready for the next launch
}

// ---------------------------------------------------------------------------------------
// Dense expansion only: lane <-> token, one ballot per row builds the packed word.
// Same grid and row groups as the fused kernel; per_split counts 32-token words here.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_expand_dense(const __grid_constant__ StepArgs a) {
    extern __shared__ __align__(128) uint32_t smem[];
    uint32_t* T = smem;
    int* s_row = reinterpret_cast<int*>(T + a.table_words);
    uint32_t* stage = reinterpret_cast<uint32_t*>(s_row + kGroupRows);

    pdl_prologue();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, n_warps = blockDim.x >> 5;
    const int g = blockIdx.x / a.S, split = blockIdx.x - g * a.S;
    if (a.n_groups && g >= __ldg(a.n_groups)) return;
    const int part = group_rows_setup(a, g, s_row, tid);
    __syncthreads();
    const PartDev P = a.group_part ? a.parts[part] : a.p0;
    const int nrow = __popc(__ballot_sync(0xFFFFFFFFu, s_row[lane] >= 0));
    if (a.stage_stride) {
        stage_class_masks(a, P, s_row, stage, warp, lane, n_warps);
        __syncthreads();
    }
    build_class_table(a, P, s_row, T, stage, warp, lane, n_warps);
    __syncthreads();

    const int w_begin = split * a.per_split, w_end = min(w_begin + a.per_split, a.VW);
    const int my_row = s_row[lane];
    uint32_t* out = a.vocab_mask + int64_t(max(my_row, 0)) * a.vm_stride;
    // a warp takes 8 consecutive words (256 tokens) per iteration; lane r ends up holding row r's words
    for (int w0 = w_begin + warp * 8; w0 < w_end; w0 += n_warps * 8) {
        uint32_t mine[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int w = w0 + q;
            uint32_t bits = 0;
            if (w < w_end) bits = T[P.c16[w * 32 + lane]];  // c16 is padded to 32*VW entries
            mine[q] = 0;
            for (int r = 0; r < nrow; ++r) {
                const uint32_t word = __ballot_sync(0xFFFFFFFFu, (bits >> r) & 1u);
                if (lane == r) mine[q] = word;
            }
        }
        if (my_row >= 0) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (w0 + q < w_end) out[w0 + q] = mine[q];
        }
    }
}

// ---------------------------------------------------------------------------------------
// Sparse step: one row per block (S blocks per row). The row's vocab bitmask is built in
// shared memory by scattering the member lists of the allowed classes; then the row is
// streamed: octets with no allowed token are overwritten with -inf without being read.
// FUSED = false stops after writing the vocab mask.
// ---------------------------------------------------------------------------------------
constexpr int kBigClass = 256;   // classes at least this large are scattered by the whole block
constexpr int kBigListCap = 64;

__device__ __forceinline__ int lower_bound_tok(const int32_t* tok, int lo, int hi, int t) {
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(tok + mid) < t) lo = mid + 1; else hi = mid;
    }
    return lo;
}

template <int DT, bool FUSED>
__global__ void __launch_bounds__(256) k_step_sparse(const __grid_constant__ StepArgs a) {
    extern __shared__ __align__(128) uint32_t smem[];
    uint32_t* bits = smem;  // per_split words
    __shared__ int s_big[kBigListCap];
    __shared__ int s_nbig;
    __shared__ int s_last;
    __shared__ Partial s_red[8];

    pdl_prologue();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, n_warps = blockDim.x >> 5;
    int row = blockIdx.x / a.S;
    const int split = blockIdx.x - row * a.S;
    __shared__ int s_batch[kBatchRows];
    if (a.row_mode) {
        // Automatic mode: the grid covers the (group, row slot) pairs of the gather kernel, and the choice is made
        // for the 8 row slots that kernel streams together (its row batch), so that no row is done twice.
        const int g = row / kGroupRows, j = row - g * kGroupRows;
        if (a.n_groups && g >= __ldg(a.n_groups)) return;
        if (tid < kBatchRows) {
            const int slot = g * kGroupRows + (j & ~(kBatchRows - 1)) + tid;
            int r = a.group_rows ? a.group_rows[slot] : slot;
            if (r >= a.B) r = -1;
            s_batch[tid] = r;
        }
        __syncthreads();
        row = s_batch[j & (kBatchRows - 1)];
        if (row < 0) return;
    }
    const int part = a.row_part ? a.row_part[row] : a.part0;
    if (part < 0 || part >= a.n_parts || !a.parts[part].live || a.parts[part].V != a.V) {
        if (tid == 0 && split == 0) atomicAdd(a.status + 2, 1);  // (never in automatic mode: only grouped rows come here)
        return;
    }
    const PartDev P = a.parts[part];
    const int w_begin = split * a.per_split, w_end = min(w_begin + a.per_split, a.VW);
    const int t0 = w_begin * 32, t1 = min(w_end * 32, a.V);
    const uint32_t* cm = a.class_mask + int64_t(row) * a.cm_stride;
    if (a.row_mode) {
        // This kernel runs first and keeps the row batches that allow few tokens (it never reads a logit that is not
        // allowed); the others it leaves, marked, to the gather kernel launched behind it. The tokens a row allows
        // are the summed sizes of its allowed classes; the rows of a batch share their partition.
        __shared__ unsigned long long s_allowed;
        if (tid == 0) s_allowed = 0ull;
        __syncthreads();
        unsigned long long mine = 0ull;
        int n_live = 0;
#pragma unroll
        for (int q = 0; q < kBatchRows; ++q) n_live += s_batch[q] >= 0;
        // a thread per class: how many of the batch's rows allow it (their mask words are the same address for the 32
        // lanes of a warp), times its size; the cost does not depend on how many classes are allowed
        for (int k = tid; k < P.K; k += blockDim.x) {
            int cnt = 0;
#pragma unroll
            for (int q = 0; q < kBatchRows; ++q) {
                const int r = s_batch[q];
                if (r >= 0) cnt += (__ldg(a.class_mask + int64_t(r) * a.cm_stride + (k >> 5)) >> (k & 31)) & 1u;
            }
            if (cnt) mine += static_cast<unsigned long long>(cnt) * static_cast<unsigned>(__ldg(P.off + k + 1) - __ldg(P.off + k));
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, d);
        if (lane == 0 && mine) atomicAdd(&s_allowed, mine);
        __syncthreads();
        const bool keep = s_allowed * 1000ull < static_cast<unsigned long long>(a.auto_permille) * unsigned(n_live) * unsigned(a.V);
        if (tid == 0 && split == 0) a.row_mode[row] = keep ? 1 : 0;
        if (!keep) return;
    }
    for (int i = tid; i < a.per_split; i += blockDim.x) bits[i] = 0u;
    if (tid == 0) s_nbig = 0;
    __syncthreads();

    for (int kw = warp; kw < P.KW; kw += n_warps) {
        uint32_t word = __ldg(cm + kw);
        if (kw == P.KW - 1 && (P.K & 31)) word &= (1u << (P.K & 31)) - 1u;
        while (word) {
            const int k = kw * 32 + __ffs(word) - 1;
            word &= word - 1u;
            int lo = __ldg(P.off + k), hi = __ldg(P.off + k + 1);
            if (a.S > 1) {
                lo = lower_bound_tok(P.tok, lo, hi, t0);
                hi = lower_bound_tok(P.tok, lo, hi, t1);
            }
            if (hi - lo >= kBigClass) {
                int slot = 0;
                if (lane == 0) slot = atomicAdd(&s_nbig, 1);
                slot = __shfl_sync(0xFFFFFFFFu, slot, 0);
                if (slot < kBigListCap) {
                    if (lane == 0) s_big[slot] = k;
                    continue;
                }
            }
            for (int i = lo + lane; i < hi; i += 4 * 32) {  // four member ids in flight per lane
                int t[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) t[q] = i + 32 * q < hi ? __ldg(P.tok + i + 32 * q) : -1;
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (t[q] >= 0) atomicOr(bits + ((t[q] >> 5) - w_begin), 1u << (t[q] & 31));
            }
        }
    }
    __syncthreads();
    const int nbig = min(s_nbig, kBigListCap);
    for (int b = 0; b < nbig; ++b) {
        const int k = s_big[b];
        int lo = __ldg(P.off + k), hi = __ldg(P.off + k + 1);
        if (a.S > 1) {
            lo = lower_bound_tok(P.tok, lo, hi, t0);
            hi = lower_bound_tok(P.tok, lo, hi, t1);
        }
        for (int i = lo + tid; i < hi; i += 4 * blockDim.x) {
            int t[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) t[q] = i + int(blockDim.x) * q < hi ? __ldg(P.tok + i + blockDim.x * q) : -1;
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (t[q] >= 0) atomicOr(bits + ((t[q] >> 5) - w_begin), 1u << (t[q] & 31));
        }
    }
    __syncthreads();

    if (a.vocab_mask) {
        uint32_t* out = a.vocab_mask + int64_t(row) * a.vm_stride;
        for (int w = w_begin + tid; w < w_end; w += blockDim.x) out[w] = bits[w - w_begin];
    }
    if (!FUSED) return;

    constexpr int ES = DT == kBF16 ? 2 : 4;
    char* rowp = reinterpret_cast<char*>(a.logits) + int64_t(row) * a.row_stride * ES;
    const uint8_t* bytes = reinterpret_cast<const uint8_t*>(bits);
    const int o_begin = 4 * w_begin, o_end = 4 * w_end, n_full = a.V >> 3;
    const int o_vec_end = min(o_end, n_full);
    RowAcc acc;
    acc.init();
    constexpr int U = 4;
    for (int ob = o_begin + tid; ob < o_vec_end; ob += U * blockDim.x) {
        Octet<DT> oc[U];
        uint32_t byte[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int o = ob + u * blockDim.x;
            byte[u] = o < o_vec_end ? bytes[o - o_begin] : 0u;
            if (byte[u]) oc[u].load(rowp, o);  // octets without an allowed token are never read
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int o = ob + u * blockDim.x;
            if (o >= o_vec_end) continue;
            if (byte[u] == 0u) {
                oc[u].fill_neg_inf();
                oc[u].store(rowp, o, a.wide != 0);
            } else {
                float f[8];
                oc[u].mask(byte[u], f);
                if (byte[u] != 0xFFu) oc[u].store(rowp, o, a.wide != 0);
                acc.add_octet(f, o);
            }
        }
    }
    // octets past the last whole vector (ragged end of the row, padding of the last mask word)
    if (o_end > n_full) {
        const int o = max(o_begin, n_full) + tid;
        if (o < o_end) {
            float f[8];
            const uint32_t byte = bytes[o - o_begin];
            octet_scalar<DT>(rowp, o, a.V, byte, f);
            if (byte) acc.add_octet(f, o);
        }
    }
    const Partial mine = acc.to_partial();
    float m = mine.m, s = mine.s;
    int pos = mine.pos;
    partial_warp_allreduce(m, s, pos);
    if (lane == 0) s_red[warp] = Partial{m, s, pos, 0};
    __threadfence();  // the row's masked logits must be visible to whichever block finishes the row
    __syncthreads();
    if (warp == 0) {
        if (lane == 0)
            for (int w = 1; w < n_warps; ++w) partial_merge(m, s, pos, s_red[w].m, s_red[w].s, s_red[w].pos);
        if (a.S == 1) {
            m = __shfl_sync(0xFFFFFFFFu, m, 0);
            s = __shfl_sync(0xFFFFFFFFu, s, 0);
            pos = __shfl_sync(0xFFFFFFFFu, pos, 0);
            warp_finalize_row<DT>(a, P, row, m, s, pos, lane);
        } else if (lane == 0) {
            a.partials[int64_t(row) * a.S + split] = Partial{m, s, pos, 0};
            __threadfence();
            s_last = (atomicAdd(a.tickets + row, 1u) == unsigned(a.S - 1));
        }
    }
    if (a.S == 1) return;
    __syncthreads();
    if (!s_last || warp != 0) return;
    __threadfence();
    float m2 = -INFINITY, s2 = 0.f;
    int p2 = kNoPos;
    for (int sp = lane; sp < a.S; sp += 32) {
        const int4 raw = __ldcg(reinterpret_cast<const int4*>(a.partials + int64_t(row) * a.S + sp));
        partial_merge(m2, s2, p2, __int_as_float(raw.x), __int_as_float(raw.y), raw.z);
    }
    partial_warp_allreduce(m2, s2, p2);
    warp_finalize_row<DT>(a, P, row, m2, s2, p2, lane);
    if (lane == 0) a.tickets[row] = 0u;
}

// ---------------------------------------------------------------------------------------
// Generic step: one block per row, one token per thread per iteration, no alignment or
// size requirement (any K, int32 class ids, odd strides). FUSED = false: expansion only.
// ---------------------------------------------------------------------------------------
template <int DT, bool FUSED>
__global__ void __launch_bounds__(256) k_step_generic(const __grid_constant__ StepArgs a) {
    __shared__ Partial s_red[8];
    pdl_prologue();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, n_warps = blockDim.x >> 5;
    const int row = blockIdx.x;
    const int part = a.row_part ? a.row_part[row] : a.part0;
    if (part < 0 || part >= a.n_parts || !a.parts[part].live || a.parts[part].V != a.V) {
        if (tid == 0) atomicAdd(a.status + 2, 1);
        return;
    }
    const PartDev P = a.parts[part];
    const uint32_t* cm = a.class_mask + int64_t(row) * a.cm_stride;
    constexpr int ES = DT == kBF16 ? 2 : 4;
    char* rowp = FUSED ? reinterpret_cast<char*>(a.logits) + int64_t(row) * a.row_stride * ES : nullptr;
    uint32_t* out = a.vocab_mask ? a.vocab_mask + int64_t(row) * a.vm_stride : nullptr;
    float m = -INFINITY, s = 0.f;
    int pos = kNoPos;
    for (int w = warp; w < a.VW; w += n_warps) {
        const int t = w * 32 + lane;
        bool allowed = false;
        if (t < a.V) {
            const int k = __ldg(P.c32 + t);
            allowed = (__ldg(cm + (k >> 5)) >> (k & 31)) & 1u;
        }
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, allowed);
        if (out && lane == 0) out[w] = word;
        if (FUSED && t < a.V) {
            if (allowed) {
                const float z = load_elem<DT>(rowp, t);
                const bool upd = (z > m) || pos == kNoPos;
                pos = upd ? t : pos;
                const float ref_old = fmaxf(m, kRefFloor);
                m = fmaxf(m, z);
                const float ref = fmaxf(m, kRefFloor);
                s = fmaf(s, ex2f((ref_old - ref) * a.scale), ex2f((z - ref) * a.scale));
            } else {
                store_neg_inf<DT>(rowp, t);
            }
        }
    }
    if (!FUSED) return;
    partial_warp_allreduce(m, s, pos, a.scale);
    if (lane == 0) s_red[warp] = Partial{m, s, pos, 0};
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < n_warps; ++w) partial_merge(m, s, pos, s_red[w].m, s_red[w].s, s_red[w].pos, a.scale);
        if (a.u)
            a.partials[row] = Partial{m, s, pos, 0};  // a sampling step: the sampling kernel takes it from here
        else
            finalize_row<DT>(a, P, row, m, s, pos, true);
    }
}

// ---------------------------------------------------------------------------------------
// Second kernel of a sampling step: one block per row draws the row's token from the tempered
// distribution over its allowed tokens by inverse CDF in token order, with the row's uniform number
// u: the lowest token whose cumulative weight exceeds u times the total. The states the streaming
// kernel published stand for consecutive runs of tokens (state k: chunks [k * run_chunks,
// (k+1) * run_chunks) of chunk_tokens tokens; with tail_state the last one: the tokens past the last whole
// vector), so the block first scans the states for the run that holds the crossing, then re-reads
// the masked logits of that run only and scans them. All sums are taken in a fixed order.
// ---------------------------------------------------------------------------------------
constexpr int kSampleThreads = 256;

// Exclusive prefix sum of one value per thread over the block, in thread order; total to everybody.
__device__ __forceinline__ float block_exclusive_scan(float v, float* s_warp, float& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const float up = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += up;
    }
    if (lane == 31) s_warp[warp] = inc;  // the caller gives every call an array no thread may still be reading
    __syncthreads();
    float before = 0.f, all = 0.f;
#pragma unroll
    for (int w = 0; w < kSampleThreads / 32; ++w) {
        const float t = s_warp[w];
        if (w < warp) before += t;
        all += t;
    }
    total = all;
    return before + inc - v;
}

template <int DT>
__global__ void __launch_bounds__(kSampleThreads) k_sample_rows(const __grid_constant__ StepArgs a, int aligned) {
    __shared__ float s_warp[kSampleThreads / 32], s_scan_states[kSampleThreads / 32], s_scan_tokens[kSampleThreads / 32];
    __shared__ int s_pick, s_last;
    __shared__ int s_pick_state, s_last_state;
    __shared__ float s_base;
    pdl_prologue();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = blockIdx.x / kGroupRows, j = blockIdx.x - g * kGroupRows;
    if (a.n_groups && g >= __ldg(a.n_groups)) return;
    int row;
    if (a.group_rows) {
        row = a.group_rows[g * kGroupRows + j];
    } else {
        row = g * kGroupRows + j;
        if (row >= a.B) row = -1;
    }
    if (row < 0) return;
    PartDev P = a.p0;
    if (a.group_part) {
        P = a.parts[a.group_part[g]];
    } else if (a.row_part) {
        const int part = a.row_part[row];
        if (part < 0 || part >= a.n_parts || !a.parts[part].live || a.parts[part].V != a.V) return;  // counted by the step kernel
        P = a.parts[part];
    }
    const Partial* src = row_slots(a, g, j);
    const float u = __ldg(a.u + row);  // needed late: in flight together with the states
    const int n_states = a.slots;
    const int per = (n_states + kSampleThreads - 1) / kSampleThreads;  // consecutive states per thread
    const int k0 = tid * per, k1 = min(k0 + per, n_states);

    // the states of this thread: fetched once, all loads in flight together, kept in registers when there are
    // at most four of them (otherwise they are fetched again wherever they are needed)
    constexpr int kKeep = 4;
    const bool kept = per <= kKeep;
    float km[kKeep], ks[kKeep];
#pragma unroll
    for (int i = 0; i < kKeep; ++i) {
        km[i] = -INFINITY;
        ks[i] = 0.f;
        if (kept && k0 + i < k1) {
            const int4 raw = __ldcg(reinterpret_cast<const int4*>(src + k0 + i));
            km[i] = __int_as_float(raw.x);
            ks[i] = __int_as_float(raw.y);
        }
    }
    // the row maximum
    float M = -INFINITY;
    if (kept) {
#pragma unroll
        for (int i = 0; i < kKeep; ++i) M = fmaxf(M, km[i]);
    } else {
        for (int k = k0; k < k1; ++k) M = fmaxf(M, __ldcg(&src[k].m));
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, d));
    if (lane == 0) s_warp[warp] = M;
    if (tid == 0) {
        s_pick = kNoPos;
        s_last = -1;
        s_pick_state = kNoPos;
        s_last_state = -1;
    }
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kSampleThreads / 32; ++w) M = fmaxf(M, s_warp[w]);
    if (!(M > kRefFloor)) {
        // nothing allowed, or only -inf allowed: the lowest allowed token (if any) and -inf logs
        if (warp == 0) {
            unsigned long long cand = first_allowed_share(a, P, row, lane, 32);
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) {
                const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, cand, d);
                cand = other < cand ? other : cand;
            }
            if (lane == 0) write_row_outputs(a, row, -INFINITY, 0.f, cand);
        }
        return;
    }

    // weights of the states relative to M, their exclusive prefix sums in token order, the total
#pragma unroll
    for (int i = 0; i < kKeep; ++i) ks[i] *= ex2f((fmaxf(km[i], kRefFloor) - M) * a.scale);  // now the weight (0 if unused)
    auto weight = [&](int k) {
        if (kept) {
            float w = 0.f;
#pragma unroll
            for (int i = 0; i < kKeep; ++i) w = (k - k0 == i) ? ks[i] : w;
            return w;
        }
        const int4 raw = __ldcg(reinterpret_cast<const int4*>(src + k));
        return __int_as_float(raw.y) * ex2f((fmaxf(__int_as_float(raw.x), kRefFloor) - M) * a.scale);
    };
    float mine = 0.f;
    for (int k = k0; k < k1; ++k) mine += weight(k);
    float total;
    const float front = block_exclusive_scan(mine, s_scan_states, total);  // weight in front of this thread's states
    const float tau = u * total;
    float run = front;
    for (int k = k0; k < k1; ++k) {
        const float w = weight(k);
        if (w > 0.f) {
            atomicMax(&s_last_state, k);
            if (run + w > tau) {
                atomicMin(&s_pick_state, k);
                break;
            }
        }
        run += w;
    }
    __syncthreads();
    // rounding may leave tau at the very end: then the last run with weight
    const int pick = s_pick_state != kNoPos ? s_pick_state : s_last_state;
    if (pick >= k0 && pick < k1) {  // the thread that owns the chosen state: the weight in front of it
        float r2 = front;
        for (int k = k0; k < pick; ++k) r2 += weight(k);
        s_base = r2;
    }
    __syncthreads();
    float base = s_base;

    // the tokens the chosen state stands for
    const int n_full8 = (a.V >> 3) << 3;
    int t_lo, t_hi;
    if (a.tail_state && pick == n_states - 1) {
        t_lo = n_full8;
        t_hi = a.V;
    } else {
        const long long lim = a.tail_state ? n_full8 : a.V;
        t_lo = int(min(static_cast<long long>(pick) * a.run_chunks * a.chunk_tokens, lim));
        t_hi = int(min(static_cast<long long>(pick + 1) * a.run_chunks * a.chunk_tokens, lim));
    }
    constexpr int ES = DT == kBF16 ? 2 : 4;
    const char* rowp = reinterpret_cast<const char*>(a.logits) + int64_t(row) * a.row_stride * ES;
    auto load8 = [&](int t0, float (&e)[8]) {
        if (aligned && t0 + 8 <= t_hi) {  // t_lo is a multiple of 8 tokens: 16-byte (bf16) / 32-byte (f32) vectors
            if (DT == kBF16) {
                const uint4 v = __ldcg(reinterpret_cast<const uint4*>(rowp + size_t(t0) * 2));
                e[0] = __uint_as_float(v.x << 16); e[1] = __uint_as_float(v.x & 0xFFFF0000u);
                e[2] = __uint_as_float(v.y << 16); e[3] = __uint_as_float(v.y & 0xFFFF0000u);
                e[4] = __uint_as_float(v.z << 16); e[5] = __uint_as_float(v.z & 0xFFFF0000u);
                e[6] = __uint_as_float(v.w << 16); e[7] = __uint_as_float(v.w & 0xFFFF0000u);
            } else {
                const float4 v0 = __ldcg(reinterpret_cast<const float4*>(rowp + size_t(t0) * 4));
                const float4 v1 = __ldcg(reinterpret_cast<const float4*>(rowp + size_t(t0) * 4 + 16));
                e[0] = v0.x; e[1] = v0.y; e[2] = v0.z; e[3] = v0.w;
                e[4] = v1.x; e[5] = v1.y; e[6] = v1.z; e[7] = v1.w;
            }
        } else {
#pragma unroll
            for (int q = 0; q < 8; ++q) e[q] = t0 + q < t_hi ? ldcg_elem<DT>(rowp, t0 + q) : -INFINITY;
        }
    };
    auto write_token = [&](int token, float zt, int repv) {
        const float l = logf(total);
        a.argmax[row] = token;
        if (a.rep) a.rep[row] = repv;
        if (a.lse) a.lse[row] = fmaf(M, a.inv_t, l);
        if (a.logp_argmax) a.logp_argmax[row] = (zt - M) * a.inv_t - l;
    };
    auto write_empty = [&]() {  // no token of the run carried weight: report the row as empty
        a.argmax[row] = -1;
        if (a.rep) a.rep[row] = -1;
        if (a.lse) a.lse[row] = -INFINITY;
        if (a.logp_argmax) a.logp_argmax[row] = -INFINITY;
    };
    if (pick < 0) {  // no state carried weight
        if (tid == 0) write_empty();
        return;
    }
    int token = -1;
    for (int p0 = t_lo; p0 < t_hi; p0 += kSampleThreads * 8) {
        const int t0 = p0 + tid * 8;
        float e[8];
        load8(t0, e);
        float z8[8], sum8 = 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            z8[q] = e[q];
            e[q] = ex2f((e[q] - M) * a.scale);  // a masked logit is -inf: weight 0
            sum8 += e[q];
        }
        float piece;
        float r3 = base + block_exclusive_scan(sum8, s_scan_tokens, piece);
        int mine_tok = -1, mine_last = -1;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            if (e[q] > 0.f && mine_tok < 0) {
                mine_last = t0 + q;
                r3 += e[q];
                if (r3 > tau) mine_tok = t0 + q;
            }
        }
        if (mine_last >= 0) atomicMax(&s_last, mine_last);
        if (mine_tok >= 0) atomicMin(&s_pick, mine_tok);
        int my_rep = mine_tok >= 0 ? __ldg(P.trep + mine_tok) : -1;  // in flight across the barrier
        __syncthreads();
        token = s_pick != kNoPos ? s_pick : -1;
        const bool last_piece = p0 + kSampleThreads * 8 >= t_hi;
        if (token < 0 && last_piece) token = s_last;  // rounding: the last token with weight in the run
        if (token >= t0 && token < t0 + 8) {          // the thread that holds the token writes the row's results
            float zt = 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q) zt = (token - t0 == q) ? z8[q] : zt;
            if (token != mine_tok) my_rep = __ldg(P.trep + token);
            write_token(token, zt, my_rep);
        }
        if (token >= 0) break;
        base += piece;
    }
    if (token < 0 && tid == 0) write_empty();
}

// ---------------------------------------------------------------------------------------
// Second kernel of a sampling step with top-k / top-p: one block per row keeps, of the row's allowed tokens in the
// order (value, largest first; equal values by token id, lowest first), the first top_k (0 = all) and of those the
// shortest beginning whose weight reaches top_p times the weight of what top_k kept (>= 1: all), then draws among
// the kept tokens by inverse CDF in token order with the row's uniform number.
// The kept set is { key > tau } plus the first m tokens, in token order, with key == tau, where key is an
// order-preserving integer image of the logit; tau is the largest key with enough tokens (top-k) or enough weight
// (top-p) at or above it. Weights are 40-bit fixed-point integers (exp((z - M) / T) * 2^40), so every sum is
// exact whatever the order of the addends: the result is deterministic. The tokens whose weight is not zero in that
// format are first collected in shared memory (up to kFiltList of them). When they all fit, which is the rule at the
// temperatures used for constrained decoding, nothing goes back to the row (a token of weight zero can change neither
// a cumulative weight nor the draw): tau, the last tie that is kept and the drawn token each come out of a radix
// search over the list, ten bits per round (list_select). Otherwise tau is found by bisection with passes over the row.
// ---------------------------------------------------------------------------------------
constexpr int kFiltThreads = 1024;
constexpr int kFiltList = 12288;  // entries of the candidate list (16 bytes each, dynamic shared memory)
constexpr int kFiltAttempts = 5;  // passes over the row with the bar for the list raised each time it overflows
constexpr int kFiltPeers = 4;     // most blocks that share a row
constexpr float kFixOne = 1099511627776.f;  // 2^40

// Order-preserving integer image of a logit and its inverse. bf16 logits only use the upper half of the float's
// bits, so their keys are 16 bits wide and a bisection over them takes half the steps.
template <int DT>
__device__ __forceinline__ uint32_t logit_key(float z) {
    z = z == 0.f ? 0.f : z;  // -0.0 and +0.0 are the same value
    const uint32_t b = __float_as_uint(z);
    const uint32_t k = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
    return DT == kBF16 ? k >> 16 : k;
}
template <int DT>
__device__ __forceinline__ float key_logit(uint32_t k) {
    if (DT == kBF16) k = (k << 16) | ((k & 0x8000u) ? 0u : 0xFFFFu);  // the lower half of a negative value's key is all ones
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}
__device__ __forceinline__ unsigned long long fixed_weight(float z, float M, float scale) {
    return __float2ull_rz(ex2f((z - M) * scale) * kFixOne);
}

struct CountMass {
    unsigned int n;
    unsigned long long w;
};

// Sum of one (count, weight) pair per thread over the block; everybody gets the total. s_n / s_w: two sets of one
// entry per warp, used in turn (`turn` flips with every call), so that one barrier per call is enough: a warp can only
// write a set again after every warp has passed the barrier of the call in between, i.e. has read this one.
__device__ __forceinline__ CountMass block_sum(CountMass v, unsigned int* s_n, unsigned long long* s_w, int& turn) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        v.n += __shfl_xor_sync(0xFFFFFFFFu, v.n, d);
        v.w += __shfl_xor_sync(0xFFFFFFFFu, v.w, d);
    }
    constexpr int kWarps = kFiltThreads / 32;
    unsigned int* n = s_n + turn * kWarps;
    unsigned long long* w = s_w + turn * kWarps;
    turn ^= 1;
    if (lane == 0) {
        n[warp] = v.n;
        w[warp] = v.w;
    }
    __syncthreads();
    CountMass t{0u, 0ull};
#pragma unroll
    for (int i = 0; i < kWarps; ++i) {
        t.n += n[i];
        t.w += w[i];
    }
    return t;
}

// Exclusive prefix sum of one 64-bit value per thread in thread order; total to everybody.
__device__ __forceinline__ unsigned long long block_exclusive_scan_u64(unsigned long long v, unsigned long long* s_w,
                                                                       unsigned long long& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += up;
    }
    __syncthreads();
    if (lane == 31) s_w[warp] = inc;
    __syncthreads();
    unsigned long long before = 0ull, all = 0ull;
#pragma unroll
    for (int w = 0; w < kFiltThreads / 32; ++w) {
        const unsigned long long t = s_w[w];
        if (w < warp) before += t;
        all += t;
    }
    total = all;
    return before + inc - v;
}

// Eight consecutive logits of a row from token t0 on (-inf past `end`), as floats.
template <int DT>
__device__ __forceinline__ void load_eight(const char* rowp, int t0, int end, bool aligned, float (&e)[8]) {
    if (aligned && t0 + 8 <= end) {
        if (DT == kBF16) {
            const uint4 v = __ldcg(reinterpret_cast<const uint4*>(rowp + size_t(t0) * 2));
            e[0] = __uint_as_float(v.x << 16); e[1] = __uint_as_float(v.x & 0xFFFF0000u);
            e[2] = __uint_as_float(v.y << 16); e[3] = __uint_as_float(v.y & 0xFFFF0000u);
            e[4] = __uint_as_float(v.z << 16); e[5] = __uint_as_float(v.z & 0xFFFF0000u);
            e[6] = __uint_as_float(v.w << 16); e[7] = __uint_as_float(v.w & 0xFFFF0000u);
        } else {
            const float4 v0 = __ldcg(reinterpret_cast<const float4*>(rowp + size_t(t0) * 4));
            const float4 v1 = __ldcg(reinterpret_cast<const float4*>(rowp + size_t(t0) * 4 + 16));
            e[0] = v0.x; e[1] = v0.y; e[2] = v0.z; e[3] = v0.w;
            e[4] = v1.x; e[5] = v1.y; e[6] = v1.z; e[7] = v1.w;
        }
    } else {
#pragma unroll
        for (int q = 0; q < 8; ++q) e[q] = t0 + q < end ? ldcg_elem<DT>(rowp, t0 + q) : -INFINITY;
    }
}

// Visit every token of a row, the block's threads side by side (8 consecutive tokens per thread and round, four
// rounds in flight together).
template <int DT, typename F>
__device__ __forceinline__ void row_visit(const char* rowp, int V, bool aligned, F&& f) {
    constexpr int kInFlight = 4;
    for (int t0 = threadIdx.x * 8; t0 < V; t0 += kFiltThreads * 8 * kInFlight) {
        float e[kInFlight][8];
#pragma unroll
        for (int r = 0; r < kInFlight; ++r) load_eight<DT>(rowp, t0 + r * kFiltThreads * 8, V, aligned, e[r]);
#pragma unroll
        for (int r = 0; r < kInFlight; ++r)
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (e[r][q] > kRefFloor) f(t0 + r * kFiltThreads * 8 + q, e[r][q]);  // masked logits are -inf
    }
}

// ---- thread-block cluster: rank, barrier, reads of a peer block's shared memory -----------------
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_blocks() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
// every thread of every block of the cluster (a hardware barrier like the block's own: no flag is polled)
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t peer_shared(const void* mine, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(mine)), "r"(rank));
    return r;
}
__device__ __forceinline__ unsigned int add_peer_u32(uint32_t addr, unsigned int v) {
    unsigned int old;
    asm volatile("atom.shared::cluster.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(addr), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ uint32_t ld_peer_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void st_peer_u64(uint32_t addr, unsigned long long v) {
    asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
}
__device__ __forceinline__ void st_peer_u32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

// ---- searches over the candidate list: every thread of the block walks the list (a walk is a chain of dependent
// shared-memory accesses per entry, so more threads shorten it), the first kSelThreads threads sum over the buckets
// (barriers and sums across 8 warps cost a fraction of those across 32)
constexpr int kSelThreads = 256;
constexpr int kSelBuckets = 1024;  // ten bits of the value per round; kSelBuckets / kSelThreads buckets per thread
__device__ __forceinline__ void sel_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kSelThreads) : "memory"); }

// Exclusive prefix of one (count, weight) pair per thread in thread order over those threads; total to everybody.
// s_n / s_w: two sets of one entry per warp, used in turn as in block_sum.
__device__ __forceinline__ CountMass sel_exclusive_scan(CountMass v, unsigned int* s_n, unsigned long long* s_w, int& turn,
                                                        CountMass& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    CountMass inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned int un = __shfl_up_sync(0xFFFFFFFFu, inc.n, d);
        const unsigned long long uw = __shfl_up_sync(0xFFFFFFFFu, inc.w, d);
        if (lane >= d) {
            inc.n += un;
            inc.w += uw;
        }
    }
    constexpr int kWarps = kSelThreads / 32;
    unsigned int* n = s_n + turn * kWarps;
    unsigned long long* w = s_w + turn * kWarps;
    turn ^= 1;
    if (lane == 31) {
        n[warp] = inc.n;
        w[warp] = inc.w;
    }
    sel_sync();
    CountMass before{0u, 0ull}, all{0u, 0ull};
#pragma unroll
    for (int i = 0; i < kWarps; ++i) {
        const unsigned int tn = n[i];
        const unsigned long long tw = w[i];
        if (i < warp) {
            before.n += tn;
            before.w += tw;
        }
        all.n += tn;
        all.w += tw;
    }
    total = all;
    return CountMass{before.n + inc.n - v.n, before.w + inc.w - v.w};
}

// Result of a search: the value found, (count, weight) of the entries below it and of the entries at it, the
// threshold that was used and (count, weight) of all entries that took part.
struct Picked {
    uint32_t x;
    CountMass before, at, all;
    unsigned long long thr;
};

// Smallest value x such that the entries of the list with value <= x together count (BY_WEIGHT: weigh) more than thr,
// where thr = thr_of(count and weight of all entries) is fixed once the first histogram is summed (so a threshold
// that depends on the total weight costs no pass of its own). xg(i, x, gn, gw) gives entry i's value (below 2^bits),
// count and weight (both 0: the entry takes no part); the caller guarantees that all entries together exceed thr.
// Ten bits of the value per round, highest first: a histogram of the round's digit over the entries that agree with
// the digits found so far, a prefix sum over the buckets, and the one bucket in which the running sum passes thr is
// the next digit. Weights are added as two 32-bit halves (the carry out of the lower half is seen in the value the
// atomic returns), which keeps every atomic a native one. Called by all threads of the block.
template <bool BY_WEIGHT, typename T, typename F>
__device__ __forceinline__ Picked list_select(unsigned int n_list, int bits, T&& thr_of, F&& xg, unsigned int* h_n,
                                              unsigned int* h_lo, unsigned int* h_hi, unsigned long long* s_pick,
                                              unsigned int* s_n, unsigned long long* s_w, int& turn) {
    const int tid = threadIdx.x;
    const int rounds = bits <= 10 ? 1 : (bits + 9) / 10;
    constexpr int kPer = kSelBuckets / kSelThreads;
    static_assert(kPer == 4 && kSelBuckets == kFiltThreads, "one bucket per thread to clear, four per summing thread");
    unsigned long long prefix = 0ull, thr = 0ull;
    CountMass carry{0u, 0ull}, at{0u, 0ull};  // carry: the entries below the digits found so far
    for (int rd = rounds - 1; rd >= 0; --rd) {
        const int shift = rd * 10;
        unsigned long long* pick = s_pick + 5 * (rd & 1);
        h_n[tid] = 0u;
        h_lo[tid] = 0u;
        h_hi[tid] = 0u;
        __syncthreads();
        if (tid == 0) {  // (what stands if no bucket qualifies: cannot happen under the caller's guarantee)
            pick[0] = 0ull;
            pick[1] = carry.n;
            pick[2] = carry.w;
            pick[3] = 0ull;
            pick[4] = 0ull;
        }
        for (unsigned int i = tid; i < n_list; i += kFiltThreads) {
            uint32_t x;
            unsigned int gn;
            unsigned long long gw;
            xg(i, x, gn, gw);
            if ((gn != 0u || gw != 0ull) && (static_cast<unsigned long long>(x) >> (shift + 10)) == prefix) {
                const uint32_t b = (x >> shift) & (kSelBuckets - 1);
                if (gn) atomicAdd(&h_n[b], gn);
                if (gw) {
                    const uint32_t lo = static_cast<uint32_t>(gw);
                    uint32_t hi = static_cast<uint32_t>(gw >> 32);
                    if (lo) {
                        const uint32_t old = atomicAdd(&h_lo[b], lo);
                        hi += (old + lo) < old ? 1u : 0u;
                    }
                    if (hi) atomicAdd(&h_hi[b], hi);
                }
            }
        }
        __syncthreads();
        if (tid < kSelThreads) {
            const uint4 vn = reinterpret_cast<const uint4*>(h_n)[tid];
            const uint4 vl = reinterpret_cast<const uint4*>(h_lo)[tid];
            const uint4 vh = reinterpret_cast<const uint4*>(h_hi)[tid];
            const CountMass h[kPer] = {{vn.x, (static_cast<unsigned long long>(vh.x) << 32) | vl.x},
                                       {vn.y, (static_cast<unsigned long long>(vh.y) << 32) | vl.y},
                                       {vn.z, (static_cast<unsigned long long>(vh.z) << 32) | vl.z},
                                       {vn.w, (static_cast<unsigned long long>(vh.w) << 32) | vl.w}};
            CountMass mine{0u, 0ull}, total;
#pragma unroll
            for (int b = 0; b < kPer; ++b) {
                mine.n += h[b].n;
                mine.w += h[b].w;
            }
            CountMass run = sel_exclusive_scan(mine, s_n, s_w, turn, total);
            if (rd == rounds - 1) {  // the first round sees every entry
                thr = thr_of(total);
                if (tid == 0) {
                    s_pick[10] = thr;
                    s_pick[11] = total.n;
                    s_pick[12] = total.w;
                }
            }
            run.n += carry.n;
            run.w += carry.w;
#pragma unroll
            for (int b = 0; b < kPer; ++b) {
                const unsigned long long below = BY_WEIGHT ? run.w : static_cast<unsigned long long>(run.n);
                const unsigned long long here = BY_WEIGHT ? h[b].w : static_cast<unsigned long long>(h[b].n);
                if (below <= thr && thr < below + here) {
                    pick[0] = static_cast<unsigned long long>(tid * kPer + b);
                    pick[1] = run.n;
                    pick[2] = run.w;
                    pick[3] = h[b].n;
                    pick[4] = h[b].w;
                }
                run.n += h[b].n;
                run.w += h[b].w;
            }
        }
        __syncthreads();
        prefix = (prefix << 10) | pick[0];
        carry = CountMass{static_cast<unsigned int>(pick[1]), pick[2]};
        at = CountMass{static_cast<unsigned int>(pick[3]), pick[4]};
    }
    return Picked{static_cast<uint32_t>(prefix), carry, at, CountMass{static_cast<unsigned int>(s_pick[11]), s_pick[12]}, s_pick[10]};
}

// One row per cluster of blocks (1, 2 or 4 of them: a short batch has fewer rows than the device has
// multiprocessors). Every block looks for the candidates in its share of the row and writes them, through the
// cluster's shared memory, into the list of the cluster's first block, which carries on alone.
template <int DT>
__global__ void __launch_bounds__(kFiltThreads) k_sample_filtered(const __grid_constant__ StepArgs a, int aligned, int top_k,
                                                                  float top_p) {
    extern __shared__ __align__(16) unsigned long long filt_smem[];
    unsigned long long* const l_w = filt_smem;                                  // kFiltList weights
    uint32_t* const l_key = reinterpret_cast<uint32_t*>(filt_smem + kFiltList);  // kFiltList keys
    int* const l_id = reinterpret_cast<int*>(l_key + kFiltList);                 // kFiltList token ids
    __shared__ unsigned int s_n[2 * kFiltThreads / 32];
    __shared__ unsigned long long s_w[2 * kFiltThreads / 32];
    __shared__ unsigned long long s_scan[kFiltThreads / 32];
    __shared__ unsigned int s_sel_n[2 * kSelThreads / 32];  // the searches' own sets (only some threads sum there, so
    __shared__ unsigned long long s_sel_w[2 * kSelThreads / 32];  // their turn must not be that of the block's sums)
    int turn_sel = 0;
    __shared__ __align__(16) unsigned int s_hn[kSelBuckets], s_hlo[kSelBuckets], s_hhi[kSelBuckets];
    __shared__ unsigned long long s_pick[16];
    __shared__ unsigned long long s_top_w[kSelThreads];  // the entries with key >= tau when there are few of them
    __shared__ uint32_t s_top_key[kSelThreads];
    __shared__ int s_top_id[kSelThreads];
    __shared__ unsigned int s_top_n;
    __shared__ float s_max[kFiltThreads / 32];
    int turn = 0;
    __shared__ unsigned int s_list_n[kFiltAttempts];  // candidates counted in each pass over the row
    __shared__ unsigned int s_low_n[kFiltPeers];      // per block of the cluster: the tokens with weight that stayed
    __shared__ unsigned long long s_low_w[kFiltPeers];  // below the bar of the last pass, and their weight
    pdl_prologue();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t n_peers = cluster_blocks(), crank = cluster_rank();
    const int slot = blockIdx.x / n_peers;  // the blocks of a cluster are neighbours along x
    const int g = slot / kGroupRows, j = slot - g * kGroupRows;
    // (every way out before the cluster's barriers depends on the row alone, so the blocks of a cluster take it together)
    if (a.n_groups && g >= __ldg(a.n_groups)) return;
    int row;
    if (a.group_rows) {
        row = a.group_rows[g * kGroupRows + j];
    } else {
        row = g * kGroupRows + j;
        if (row >= a.B) row = -1;
    }
    if (row < 0) return;
    PartDev P = a.p0;
    if (a.group_part) {
        P = a.parts[a.group_part[g]];
    } else if (a.row_part) {
        const int part = a.row_part[row];
        if (part < 0 || part >= a.n_parts || !a.parts[part].live || a.parts[part].V != a.V) return;  // counted by the step kernel
        P = a.parts[part];
    }
    // the row maximum from the states the streaming kernel published
    const Partial* src = row_slots(a, g, j);
    float M = -INFINITY;
    for (int k = tid; k < a.slots; k += kFiltThreads) M = fmaxf(M, __ldcg(&src[k].m));
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, d));
    if (lane == 0) s_max[warp] = M;
    if (tid < kFiltAttempts) s_list_n[tid] = 0u;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kFiltThreads / 32; ++w) M = fmaxf(M, s_max[w]);
    if (!(M > kRefFloor)) {
        // nothing allowed, or only -inf allowed: the lowest allowed token (if any) and -inf logs
        if (warp == 0 && crank == 0) {
            unsigned long long cand = first_allowed_share(a, P, row, lane, 32);
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) {
                const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, cand, d);
                cand = other < cand ? other : cand;
            }
            if (lane == 0) write_row_outputs(a, row, -INFINITY, 0.f, cand);
        }
        return;
    }
    constexpr int ES = DT == kBF16 ? 2 : 4;
    const char* rowp = reinterpret_cast<const char*>(a.logits) + int64_t(row) * a.row_stride * ES;
    const float scale = a.scale;
    const uint32_t key_max = logit_key<DT>(M);
    // The candidates are the tokens at or above M - 41 / scale (below M - 40 / scale the fixed-point weight is zero;
    // the extra unit covers the rounding of the threshold itself). The candidates of every block go straight into the
    // list of the cluster's first block (places are reserved in its counter, a warp at a time). A comparison of
    // floats decides (z_cut is the lowest logit whose key reaches key_list), and a round of eight logits is skipped as
    // soon as its maximum falls short. When the list overflows (a flat row, or a mask that allows most of the
    // vocabulary) the row is gone over again with the bar half as far below M; what carries weight below the bar is
    // then only counted and summed (low): enough as long as top-k and top-p end inside the list.
    const float z_zero = key_logit<DT>(logit_key<DT>(M - 41.f / scale));
    uint32_t key_list = 0u;
    unsigned int n_list = 0u;
    int attempt = 0;
    {
        const uint32_t list_key0 = peer_shared(l_key, 0u), list_id0 = peer_shared(l_id, 0u);
        const int share = ((a.V + int(n_peers) - 1) / int(n_peers) + 7) & ~7;
        const int t_begin = min(int(crank) * share, a.V), t_end = min(t_begin + share, a.V);
        constexpr int kInFlight = 4;
        float units = 41.f;
        cluster_barrier();  // the first block's counters are cleared before anybody adds to them
        for (;; ++attempt, units *= 0.5f) {
            key_list = logit_key<DT>(M - units / scale);
            const float z_cut = key_logit<DT>(key_list);
            const uint32_t list_n0 = peer_shared(&s_list_n[attempt], 0u);
            CountMass low{0u, 0ull};
            // (the loop bound is the same for the lanes of a warp: they reserve their places in the list together)
            for (int tw = t_begin + warp * 256; tw < t_end; tw += kFiltThreads * 8 * kInFlight) {
                const int t0 = tw + lane * 8;
                float e[kInFlight][8];
#pragma unroll
                for (int r = 0; r < kInFlight; ++r) load_eight<DT>(rowp, t0 + r * kFiltThreads * 8, t_end, aligned != 0, e[r]);
                uint32_t cand = 0u;  // bit 8 r + q: logit q of round r is a candidate
#pragma unroll
                for (int r = 0; r < kInFlight; ++r) {
                    const float top = fmax3(fmax3(e[r][0], e[r][1], e[r][2]), fmax3(e[r][3], e[r][4], e[r][5]), fmaxf(e[r][6], e[r][7]));
                    if (top >= z_cut) {
#pragma unroll
                        for (int q = 0; q < 8; ++q) cand |= e[r][q] >= z_cut ? 1u << (8 * r + q) : 0u;
                    }
                    if (attempt > 0 && top >= z_zero) {
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            if (e[r][q] >= z_zero && e[r][q] < z_cut) {
                                low.n += 1u;
                                low.w += fixed_weight(e[r][q], M, scale);
                            }
                    }
                }
                const int cnt = __popc(cand);
                int inc = cnt;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const int up = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                    if (lane >= d) inc += up;
                }
                const int warp_cnt = __shfl_sync(0xFFFFFFFFu, inc, 31);
                if (warp_cnt == 0) continue;
                unsigned int base = 0u;
                if (lane == 31) base = add_peer_u32(list_n0, unsigned(warp_cnt));
                base = __shfl_sync(0xFFFFFFFFu, base, 31);
                unsigned int at = base + unsigned(inc - cnt);
#pragma unroll
                for (int r = 0; r < kInFlight; ++r)
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        if ((cand >> (8 * r + q)) & 1u) {
                            if (at < kFiltList) {  // (key and weight follow below, for the listed logits only)
                                st_peer_u32(list_key0 + at * 4u, __float_as_uint(e[r][q]));
                                st_peer_u32(list_id0 + at * 4u, uint32_t(t0 + r * kFiltThreads * 8 + q));
                            }
                            ++at;
                        }
            }
            if (attempt > 0) {
                const CountMass mine = block_sum(low, s_n, s_w, turn);
                if (tid == 0) {
                    st_peer_u32(peer_shared(&s_low_n[crank], 0u), mine.n);
                    st_peer_u64(peer_shared(&s_low_w[crank], 0u), mine.w);
                }
            }
            cluster_barrier();  // every block's candidates have arrived
            n_list = ld_peer_u32(list_n0);
            if (n_list <= kFiltList || attempt == kFiltAttempts - 1) break;  // (the same in every block of the cluster)
        }
    }
    if (crank != 0u) return;  // (the first block touches no other block's memory from here on)
    for (unsigned int i = tid; i < min(n_list, unsigned(kFiltList)); i += kFiltThreads) {
        const float z = __uint_as_float(l_key[i]);
        l_key[i] = logit_key<DT>(z);
        l_w[i] = fixed_weight(z, M, scale);
    }
    __syncthreads();
    const bool list_whole = n_list <= kFiltList;
    CountMass low{0u, 0ull};  // what carries weight and is not in the list
    if (attempt > 0)
        for (uint32_t p = 0; p < n_peers; ++p) {
            low.n += s_low_n[p];
            low.w += s_low_w[p];
        }

    // kept: { key > tau } and the first m tokens, in token order, with key == tau; S their weight
    uint32_t tau = 0u;
    unsigned int m = 0xFFFFFFFFu;

    if (list_whole) do {
        // ---- everything from the list (it holds the tokens that carry weight, or the heaviest of them, in no
        // particular order); leaves for the passes over the row below when top-k or top-p reach past the list
        auto select = [&](auto kind, int bits, auto&& thr_of, auto&& xg) {
            return list_select<decltype(kind)::value>(n_list, bits, thr_of, xg, s_hn, s_hlo, s_hhi, s_pick, s_sel_n, s_sel_w, turn_sel);
        };
        const std::integral_constant<bool, false> by_count;
        const std::integral_constant<bool, true> by_weight;
        // keys from the top: x = key_max - key, below 2^key_bits
        const int key_bits = 32 - __clz(key_max - key_list);
        auto from_top = [&](unsigned int i, uint32_t& x, unsigned int& gn, unsigned long long& gw) {
            x = key_max - l_key[i];
            gn = 1u;
            gw = l_w[i];
        };
        // the target of top-p: that share of the weight kept so far, rounded up; at least one unit so that one token is kept
        auto target_of = [&](unsigned long long S) {
            const unsigned long long t = static_cast<unsigned long long>(ceil(static_cast<double>(S) * static_cast<double>(top_p)));
            return t < 1ull ? 1ull : (t > S ? S : t);
        };
        unsigned long long S = 0ull;        // weight of what is kept so far (once something has been cut)
        unsigned long long w_above = 0ull;  // weight of the tokens with key > tau
        unsigned int n_above = 0u;          // their number
        unsigned int n_ties = 0u;           // tokens with key == tau
        unsigned long long w_tie = 0ull;    // weight of each of them
        bool cut = false;
        // (a top_k beyond everything that carries weight only adds tokens of weight zero: nothing to do)
        if (top_k > 0 && unsigned(top_k) >= n_list && unsigned(top_k) - n_list < low.n) break;  // ends below the list
        if (top_k > 0 && unsigned(top_k) < n_list) {
            // the largest key with at least top_k entries at or above it
            const Picked pk = select(by_count, key_bits, [&](CountMass) { return static_cast<unsigned long long>(top_k) - 1ull; },
                                     from_top);
            tau = key_max - pk.x;
            m = unsigned(top_k) - pk.before.n;
            n_ties = pk.at.n;
            w_tie = fixed_weight(key_logit<DT>(tau), M, scale);
            w_above = pk.before.w;
            n_above = pk.before.n;
            S = w_above + static_cast<unsigned long long>(m) * w_tie;
            cut = true;
        }
        if (top_p < 1.f) {
            const unsigned long long target = cut ? target_of(S) : 0ull;
            if (!cut || w_above >= target) {
                // the largest key whose entries, with those above it, reach the target (without a cut so far the target
                // follows from the weight of the whole list, which the search sums on its way)
                const Picked pk = select(by_weight, key_bits,
                                         [&](CountMass all) { return (cut ? target : target_of(all.w + low.w)) - 1ull; }, from_top);
                const unsigned long long tgt = pk.thr + 1ull;
                if (pk.all.w < tgt) break;  // the list does not hold the target (only possible with tokens left below it)
                tau = key_max - pk.x;
                w_tie = fixed_weight(key_logit<DT>(tau), M, scale);
                w_above = pk.before.w;
                n_above = pk.before.n;
                n_ties = pk.at.n;
                unsigned int need = n_ties;  // all the ties unless fewer reach the target
                if (w_tie > 0ull) {
                    const unsigned long long q = (tgt - w_above + w_tie - 1ull) / w_tie;
                    if (q < need) need = unsigned(q);
                }
                m = need < 1u ? 1u : need;
                cut = true;
            } else if (w_tie > 0ull) {
                // the target is reached among the ties at tau itself
                const unsigned long long q = (target - w_above + w_tie - 1ull) / w_tie;
                if (q < m) m = unsigned(q < 1ull ? 1ull : q);
            }
        }
        // The ties that are kept are those with the m lowest ids; the drawn token is the lowest id t with
        // (kept weight at ids <= t) > floor(u * kept weight). All ties weigh the same, so the kept weight needs no pass.
        if (!cut && low.n > 0u) break;  // nothing is cut away: the draw is over the whole row
        const float u = __ldg(a.u + row);
        auto threshold_of = [&](unsigned long long S_kept) {  // (S_kept > 0: the row maximum is always kept)
            const unsigned long long t = static_cast<unsigned long long>(static_cast<double>(u) * static_cast<double>(S_kept));
            return t >= S_kept ? S_kept - 1ull : t;
        };
        if (cut && n_above + n_ties <= unsigned(kSelThreads)) {
            // Few tokens at or above tau (the rule with top-k, and with top-p on a peaked distribution): one per thread,
            // and every thread sums over all of them: the ties below its id for its rank, the kept weight up to its id
            // for its place in the cumulative distribution.
            const unsigned long long S_kept = w_above + static_cast<unsigned long long>(min(m, n_ties)) * w_tie;
            const unsigned long long thr = threshold_of(S_kept);
            const unsigned int n_top = n_above + n_ties;
            if (tid == 0) s_top_n = 0u;
            __syncthreads();
            for (unsigned int i = tid; i < n_list; i += kFiltThreads)
                if (l_key[i] >= tau) {
                    const unsigned int at = atomicAdd(&s_top_n, 1u);
                    s_top_key[at] = l_key[i];
                    s_top_id[at] = l_id[i];
                    s_top_w[at] = l_w[i];
                }
            __syncthreads();
            if (tid >= kSelThreads) return;
            const bool have = unsigned(tid) < n_top;
            const int my_id = have ? s_top_id[tid] : a.V;
            const uint32_t my_key = have ? s_top_key[tid] : 0u;
            unsigned long long my_w = have ? s_top_w[tid] : 0ull;
            if (m < n_ties) {
                unsigned int rank = 0u;
                for (unsigned int k = 0; k < n_top; ++k) rank += (s_top_key[k] == tau && s_top_id[k] < my_id) ? 1u : 0u;
                if (have && my_key == tau && rank >= m) {
                    my_w = 0ull;
                    s_top_w[tid] = 0ull;  // (read by the others only after the barrier below)
                }
            }
            sel_sync();
            unsigned long long cum = 0ull;
            for (unsigned int k = 0; k < n_top; ++k) cum += s_top_id[k] <= my_id ? s_top_w[k] : 0ull;
            if (my_w > 0ull && cum - my_w <= thr && thr < cum) {  // the one thread that holds the drawn token
                const float l = logf(static_cast<float>(S_kept) * (1.f / kFixOne));
                const float zt = key_logit<DT>(my_key);
                a.argmax[row] = my_id;
                if (a.rep) a.rep[row] = __ldg(P.trep + my_id);
                if (a.lse) a.lse[row] = fmaf(M, a.inv_t, l);
                if (a.logp_argmax) a.logp_argmax[row] = (zt - M) * a.inv_t - l;
            }
            return;
        }
        const int id_bits = 32 - __clz(max(a.V - 1, 1));
        int id_cut = a.V;  // the kept ties are those with ids up to id_cut
        if (cut && m < n_ties)
            id_cut = int(select(by_count, id_bits, [&](CountMass) { return static_cast<unsigned long long>(m) - 1ull; },
                                [&](unsigned int i, uint32_t& x, unsigned int& gn, unsigned long long& gw) {
                                    x = uint32_t(l_id[i]);
                                    gn = l_key[i] == tau ? 1u : 0u;
                                    gw = 0ull;
                                })
                             .x);
        // (the kept weight is the weight of everything that takes part in the search for the token)
        const Picked drawn = select(by_weight, id_bits, [&](CountMass all) { return threshold_of(all.w); },
                                    [&](unsigned int i, uint32_t& x, unsigned int& gn, unsigned long long& gw) {
                                        const uint32_t key = l_key[i];
                                        const int id = l_id[i];
                                        x = uint32_t(id);
                                        gn = 0u;
                                        gw = (!cut || key > tau || (key == tau && id <= id_cut)) ? l_w[i] : 0ull;
                                    });
        const int token = int(drawn.x);
        const float l = logf(static_cast<float>(drawn.all.w) * (1.f / kFixOne));
        for (unsigned int i = tid; i < n_list; i += kFiltThreads)
            if (l_id[i] == token) {  // the one thread that holds the drawn token writes the row's results
                const float zt = key_logit<DT>(l_key[i]);
                a.argmax[row] = token;
                if (a.rep) a.rep[row] = __ldg(P.trep + token);
                if (a.lse) a.lse[row] = fmaf(M, a.inv_t, l);
                if (a.logp_argmax) a.logp_argmax[row] = (zt - M) * a.inv_t - l;
            }
        return;
    } while (false);

    // ---- the list does not reach (a flat distribution): counts and weights come from passes over the row, tau by
    // bisection on the key
    tau = 0u;
    m = 0xFFFFFFFFu;
    auto above = [&](uint32_t lo) {  // (count, weight) of the tokens with key >= lo
        CountMass v{0u, 0ull};
        row_visit<DT>(rowp, a.V, aligned != 0, [&](int, float z) {
            if (logit_key<DT>(z) >= lo) {
                v.n += 1u;
                v.w += fixed_weight(z, M, scale);
            }
        });
        return block_sum(v, s_n, s_w, turn);
    };
    const CountMass all = above(0u);
    unsigned long long S = all.w;
    if (top_k > 0 && unsigned(top_k) < all.n) {
        uint32_t lo = 0u, hi = key_max;  // count(>= lo) >= top_k holds
        while (lo < hi) {
            const uint32_t mid = lo + (hi - lo + 1u) / 2u;
            if (above(mid).n >= unsigned(top_k)) lo = mid; else hi = mid - 1u;
        }
        tau = lo;
        const CountMass gt = tau == key_max ? CountMass{0u, 0ull} : above(tau + 1u);
        m = unsigned(top_k) - gt.n;
        S = gt.w + static_cast<unsigned long long>(m) * fixed_weight(key_logit<DT>(tau), M, scale);
    }
    if (top_p < 1.f) {
        unsigned long long target = static_cast<unsigned long long>(ceil(static_cast<double>(S) * static_cast<double>(top_p)));
        target = target < 1ull ? 1ull : (target > S ? S : target);
        const CountMass gt_tau = tau >= key_max ? CountMass{0u, 0ull} : above(tau + 1u);
        if (gt_tau.w >= target) {
            uint32_t lo = tau + 1u, hi = key_max;  // weight(>= lo) >= target holds
            while (lo < hi) {
                const uint32_t mid = lo + (hi - lo + 1u) / 2u;
                if (above(mid).w >= target) lo = mid; else hi = mid - 1u;
            }
            const CountMass ge = above(lo);
            const CountMass gt = lo == key_max ? CountMass{0u, 0ull} : above(lo + 1u);
            const unsigned long long w_tie = fixed_weight(key_logit<DT>(lo), M, scale);
            unsigned int need = ge.n - gt.n;
            if (w_tie > 0ull) {
                const unsigned long long q = (target - gt.w + w_tie - 1ull) / w_tie;
                if (q < need) need = unsigned(q);
            }
            tau = lo;
            m = need < 1u ? 1u : need;
        } else {
            const unsigned long long w_tie = fixed_weight(key_logit<DT>(tau), M, scale);
            if (w_tie > 0ull) {
                const unsigned long long q = (target - gt_tau.w + w_tie - 1ull) / w_tie;
                if (q < m) m = unsigned(q < 1ull ? 1ull : q);
            }
        }
    }

    // Draw in token order. Every thread owns one contiguous segment of the row: first the ties per segment (their
    // rank decides which of them are kept), then the kept weight per segment, then the one thread whose segment
    // holds the crossing walks it once more.
    const int seg = ((a.V + kFiltThreads - 1) / kFiltThreads + 7) & ~7;
    const int t_lo = min(tid * seg, a.V), t_hi = min(t_lo + seg, a.V);
    auto seg_visit = [&](auto&& f) {
        for (int t0 = t_lo; t0 < t_hi; t0 += 32) {
            float e[4][8];
#pragma unroll
            for (int r = 0; r < 4; ++r) load_eight<DT>(rowp, t0 + 8 * r, t_hi, aligned != 0, e[r]);
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (e[r][q] > kRefFloor) f(t0 + 8 * r + q, e[r][q]);
        }
    };
    unsigned long long my_ties = 0ull;
    seg_visit([&](int, float z) { my_ties += logit_key<DT>(z) == tau ? 1ull : 0ull; });
    unsigned long long total_ties;
    const unsigned long long tie_base = block_exclusive_scan_u64(my_ties, s_scan, total_ties);
    unsigned long long my_w = 0ull, ties_seen = tie_base;
    seg_visit([&](int, float z) {
        const uint32_t key = logit_key<DT>(z);
        if (key > tau || (key == tau && ties_seen++ < m)) my_w += fixed_weight(z, M, scale);
    });
    unsigned long long S_drawn;
    const unsigned long long w_base = block_exclusive_scan_u64(my_w, s_scan, S_drawn);
    // u * S rounded down: the first token whose cumulative weight exceeds it is drawn
    const float u = __ldg(a.u + row);
    unsigned long long thr = static_cast<unsigned long long>(static_cast<double>(u) * static_cast<double>(S_drawn));
    if (S_drawn > 0ull && thr >= S_drawn) thr = S_drawn - 1ull;
    if (S_drawn == 0ull) {  // cannot happen while the row maximum is kept; reported as an empty row
        if (tid == 0) {
            a.argmax[row] = -1;
            if (a.rep) a.rep[row] = -1;
            if (a.lse) a.lse[row] = -INFINITY;
            if (a.logp_argmax) a.logp_argmax[row] = -INFINITY;
        }
        return;
    }
    if (my_w > 0ull && w_base <= thr && thr < w_base + my_w) {
        unsigned long long cum = w_base;
        int token = -1;
        float zt = 0.f;
        ties_seen = tie_base;
        seg_visit([&](int t, float z) {
            const uint32_t key = logit_key<DT>(z);
            if (key > tau || (key == tau && ties_seen++ < m)) {
                cum += fixed_weight(z, M, scale);
                if (token < 0 && cum > thr) {
                    token = t;
                    zt = z;
                }
            }
        });
        const float l = logf(static_cast<float>(S_drawn) * (1.f / kFixOne));
        a.argmax[row] = token;
        if (a.rep) a.rep[row] = token >= 0 ? __ldg(P.trep + token) : -1;
        if (a.lse) a.lse[row] = fmaf(M, a.inv_t, l);
        if (a.logp_argmax) a.logp_argmax[row] = (zt - M) * a.inv_t - l;
    }
}

// ---------------------------------------------------------------------------------------
// Row-split step on caller-provided tables: the per-row kernel above, with each row shared by
// S blocks that meet through a scratch area of (max, sum-exp, token) states and one ticket
// per row, exactly as the sparse kernel's blocks do. It touches no context: token->class and
// class->representative vectors, masks, logits and outputs all come from the caller, the
// scratch area from whoever launches it.
// ---------------------------------------------------------------------------------------
struct RowSplitArgs {
    const int32_t* c;   // dev [V]
    const int32_t* r;   // dev [K]
    int32_t V, K, VW;
    const uint32_t* class_mask;
    int64_t cm_stride;
    void* logits;
    int64_t row_stride;
    uint32_t* vocab_mask;  // nullable
    int64_t vm_stride;
    int32_t* argmax;
    int32_t* rep;          // nullable
    float* logp_argmax;    // nullable
    float* lse;            // nullable
    int32_t B, S, words_per_split;
    Partial* partials;     // [B * S]
    unsigned int* tickets; // [B], zero on entry, left zero
};

template <int DT>
__global__ void __launch_bounds__(256) k_step_rowsplit(const __grid_constant__ RowSplitArgs a) {
    __shared__ Partial s_red[8];
    __shared__ int s_last;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, n_warps = blockDim.x >> 5;
    const int row = blockIdx.x / a.S, split = blockIdx.x - row * a.S;
    const uint32_t* cm = a.class_mask + int64_t(row) * a.cm_stride;
    constexpr int ES = DT == kBF16 ? 2 : 4;
    char* rowp = reinterpret_cast<char*>(a.logits) + int64_t(row) * a.row_stride * ES;
    uint32_t* out = a.vocab_mask ? a.vocab_mask + int64_t(row) * a.vm_stride : nullptr;
    const int w_begin = split * a.words_per_split, w_end = min(w_begin + a.words_per_split, a.VW);
    float m = -INFINITY, s = 0.f;
    int pos = kNoPos;
    for (int w = w_begin + warp; w < w_end; w += n_warps) {
        const int t = w * 32 + lane;
        bool allowed = false;
        if (t < a.V) {
            const int k = __ldg(a.c + t);
            if (k >= 0 && k < a.K) allowed = (__ldg(cm + (k >> 5)) >> (k & 31)) & 1u;  // ids out of range: not allowed
        }
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, allowed);
        if (out && lane == 0) out[w] = word;
        if (t < a.V) {
            if (allowed) {
                const float z = load_elem<DT>(rowp, t);
                const bool upd = (z > m) || pos == kNoPos;
                pos = upd ? t : pos;
                const float ref_old = fmaxf(m, kRefFloor);
                m = fmaxf(m, z);
                const float ref = fmaxf(m, kRefFloor);
                s = fmaf(s, ex2f((ref_old - ref) * kLog2e), ex2f((z - ref) * kLog2e));
            } else {
                store_neg_inf<DT>(rowp, t);
            }
        }
    }
    partial_warp_allreduce(m, s, pos);
    if (lane == 0) s_red[warp] = Partial{m, s, pos, 0};
    __syncthreads();
    if (warp != 0) return;
    if (lane == 0)
        for (int w = 1; w < n_warps; ++w) partial_merge(m, s, pos, s_red[w].m, s_red[w].s, s_red[w].pos);
    if (a.S > 1) {
        if (lane == 0) {
            a.partials[int64_t(row) * a.S + split] = Partial{m, s, pos, 0};
            __threadfence();
            s_last = (atomicAdd(a.tickets + row, 1u) == unsigned(a.S - 1));
        }
        __syncwarp();
        if (!s_last) return;
        __threadfence();
        m = -INFINITY; s = 0.f; pos = kNoPos;
        for (int sp = lane; sp < a.S; sp += 32) {
            const int4 raw = __ldcg(reinterpret_cast<const int4*>(a.partials + int64_t(row) * a.S + sp));
            partial_merge(m, s, pos, __int_as_float(raw.x), __int_as_float(raw.y), raw.z);
        }
        partial_warp_allreduce(m, s, pos);
        if (lane == 0) a.tickets[row] = 0u;
    }
    if (lane != 0) return;
    int tok = -1, repv = -1;
    float lsev = -INFINITY, lpa = -INFINITY;
    if (pos != kNoPos) {
        tok = pos;
        const int k = a.c[tok];
        repv = a.r[k];
        if (m > kRefFloor && s > 0.f) {
            const float l = logf(s);
            lsev = m + l;
            lpa = -l;
        }
    }
    a.argmax[row] = tok;
    if (a.rep) a.rep[row] = repv;
    if (a.lse) a.lse[row] = lsev;
    if (a.logp_argmax) a.logp_argmax[row] = lpa;
}

// ---------------------------------------------------------------------------------------
// Row plan for batches that mix partitions: bucket the rows by partition into groups of
// up to 32 rows (valid slots first). One block.
// ---------------------------------------------------------------------------------------
constexpr int kMaxParts = 256;

__global__ void __launch_bounds__(1024) k_plan_rows(const PartDev* parts, int n_parts, const int32_t* row_part, int B,
                                                    int V, int max_groups, int32_t* group_part, int32_t* group_rows,
                                                    int32_t* n_groups, int32_t* status) {
    __shared__ int cnt[kMaxParts], gbase[kMaxParts + 1], cur[kMaxParts];
    pdl_prologue();
    const int tid = threadIdx.x;
    for (int p = tid; p < kMaxParts; p += blockDim.x) { cnt[p] = 0; cur[p] = 0; }
    __syncthreads();
    for (int b = tid; b < B; b += blockDim.x) {
        const int p = row_part[b];
        if (p >= 0 && p < n_parts && parts[p].live && parts[p].V == V) atomicAdd(&cnt[p], 1);
        else atomicAdd(status + 2, 1);
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        for (int p = 0; p < n_parts; ++p) { gbase[p] = acc; acc += (cnt[p] + kGroupRows - 1) / kGroupRows; }
        gbase[n_parts] = acc;
        *n_groups = acc;
    }
    __syncthreads();
    const int total = gbase[n_parts];
    for (int i = tid; i < max_groups * kGroupRows; i += blockDim.x) group_rows[i] = -1;
    for (int p = 0; p < n_parts; ++p)
        for (int gq = gbase[p] + tid; gq < gbase[p + 1]; gq += blockDim.x) group_part[gq] = p;
    for (int gq = total + tid; gq < max_groups; gq += blockDim.x) group_part[gq] = 0;
    __syncthreads();
    for (int b = tid; b < B; b += blockDim.x) {
        const int p = row_part[b];
        if (p >= 0 && p < n_parts && parts[p].live && parts[p].V == V) {
            const int slot = atomicAdd(&cur[p], 1);
            group_rows[(gbase[p] + slot / kGroupRows) * kGroupRows + (slot % kGroupRows)] = b;
        }
    }
}

// ---------------------------------------------------------------------------------------
// mask_logits: apply an existing vocab bitmask in place. Octets whose 8 tokens are all
// allowed are neither read nor written; octets with none allowed are written without a read.
// ---------------------------------------------------------------------------------------
template <int DT, bool ALIGNED>
__global__ void __launch_bounds__(256) k_mask_logits(void* logits, int64_t row_stride, int B, int V, int VW,
                                                     const uint32_t* vocab_mask, int64_t vm_stride, int wide) {
    pdl_prologue();
    constexpr int ES = DT == kBF16 ? 2 : 4;
    constexpr int U = 4;
    const int n_octets = (V + 7) >> 3, n_full = V >> 3;
    const int chunks = (n_octets + blockDim.x * U - 1) / (blockDim.x * U);
    const int64_t total = int64_t(B) * chunks;
    const uint8_t* vm8 = reinterpret_cast<const uint8_t*>(vocab_mask);
    for (int64_t item = blockIdx.x; item < total; item += gridDim.x) {
        const int row = int(item / chunks), ch = int(item - int64_t(row) * chunks);
        char* rowp = reinterpret_cast<char*>(logits) + int64_t(row) * row_stride * ES;
        const uint8_t* vrow = vm8 + int64_t(row) * vm_stride * 4;
        const int ob = ch * blockDim.x * U + threadIdx.x;
        Octet<DT> oc[U];
        uint32_t byte[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int o = ob + u * blockDim.x;
            byte[u] = 0xFFu;
            if (o < n_octets) {
                byte[u] = vrow[o];
                if (8 * o + 8 > V) byte[u] = (byte[u] | (0xFFu << (V - 8 * o))) & 0xFFu;  // past V: leave alone
                if (ALIGNED && o < n_full && byte[u] != 0xFFu && byte[u] != 0u) oc[u].load(rowp, o);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int o = ob + u * blockDim.x;
            if (o >= n_octets || byte[u] == 0xFFu) continue;
            float f[8];
            if (ALIGNED && o < n_full) {
                if (byte[u] == 0u) oc[u].fill_neg_inf(); else oc[u].mask(byte[u], f);
                oc[u].store(rowp, o, wide != 0);
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (8 * o + j < V && !((byte[u] >> j) & 1u)) store_neg_inf<DT>(rowp, 8 * o + j);
            }
        }
    }
}

// Measurement aid: the cheapest in-place read-modify-write over a logits matrix (every whole 16-byte vector of
// every row is read, the sign bits of its elements are flipped, and it is written back). It moves the bytes a
// step must at least move and does nothing else, so its time under the same launch protocol is what the
// step's time is compared with.
template <int DT>
__global__ void __launch_bounds__(256) k_rmw_floor(void* logits, int64_t row_stride, int B, int V) {
    pdl_prologue();
    constexpr int ES = DT == kBF16 ? 2 : 4;
    constexpr int U = 4;
    constexpr uint32_t kSign = DT == kBF16 ? 0x80008000u : 0x80000000u;
    const int nvec = int((int64_t(V) * ES) >> 4);
    const int chunks = (nvec + 256 * U - 1) / (256 * U);
    const int64_t total = int64_t(B) * chunks;
    for (int64_t item = blockIdx.x; item < total; item += gridDim.x) {
        const int row = int(item / chunks), ch = int(item - int64_t(row) * chunks);
        char* rowp = reinterpret_cast<char*>(logits) + int64_t(row) * row_stride * ES;
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = ch * 256 * U + u * 256 + threadIdx.x;
            if (i < nvec) v[u] = ld_stream16(rowp + size_t(i) * 16);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int i = ch * 256 * U + u * 256 + threadIdx.x;
            if (i < nvec) {
                v[u].x ^= kSign; v[u].y ^= kSign; v[u].z ^= kSign; v[u].w ^= kSign;
                st_stream16(rowp + size_t(i) * 16, v[u]);
            }
        }
    }
}

// logp_full[b, i] = z'[b, i] - lse[b] from the masked logits (fp32 out, row stride V).
template <int DT>
__global__ void __launch_bounds__(256) k_logp_full(const void* logits, int64_t row_stride, int B, int V, const float* lse,
                                                   float* out) {
    pdl_prologue();
    // grid: x strides over the tokens of a row, y over the rows
    for (int row = blockIdx.y; row < B; row += gridDim.y) {
        const float l = lse[row];
        for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < V; t += gridDim.x * blockDim.x) {
            const float z = load_elem<DT>(logits, int64_t(row) * row_stride + t);
            out[int64_t(row) * V + t] = (l == -INFINITY || z == -INFINITY) ? -INFINITY : z - l;
        }
    }
}

// reps[b] = r[c[tokens[b]]]
__global__ void __launch_bounds__(256) k_map_tokens(const PartDev* parts, int n_parts, int part0, const int32_t* row_part,
                                                    const int32_t* tokens, int32_t* reps, int B, int V_expected,
                                                    int32_t* status) {
    pdl_prologue();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int p = row_part ? row_part[b] : part0;
    if (p < 0 || p >= n_parts || !parts[p].live || parts[p].V != V_expected) {
        atomicAdd(status + 2, 1);
        return;
    }
    const int t = tokens[b];
    int rv = -1;
    if (t >= 0 && t < parts[p].V) rv = parts[p].trep[t];
    else atomicAdd(status + 1, 1);
    reps[b] = rv;
}

}  // namespace cfgzip
