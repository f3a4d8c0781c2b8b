// Offline step of CFGzip behind the C ABI (declarations and contracts: include/cfgzip.h).
//   host: grammars in Greibach normal form, the stack-adjacency relation (Appendix C), the displacement of every
//         token (Algorithm 1) serialised into fixed-width signature rows;
//   GPU : grouping of tokens with equal signature into classes, representatives, class lists (Section 3.1,
//         "Pre-Computation").
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <new>
#include <set>
#include <utility>
#include <vector>

#include "cfgzip.h"

struct cfgzip_grammar {
    int32_t n = 0, start = 0;
    struct Prod {
        int32_t head;
        uint8_t term;
        std::vector<int32_t> rhs;
    };
    std::vector<Prod> prods;
    std::vector<std::vector<int32_t>> by_term;  // production indices by terminal byte
    std::vector<uint8_t> adj;                   // n * n, adj[y * n + z] = 1: z may be popped right after y left nothing
};

namespace {

using Stack = std::vector<int32_t>;
using Pair = std::pair<Stack, Stack>;  // (input queue, output stack: top first)

// Appendix C: edge A -> B for every production whose right-most non-terminal is B; for every production
// A -> a B_1 .. B_n Z beta a breadth-first search from B_n collects the reachable Y with a production Y -> y.
void build_adjacency(cfgzip_grammar& g) {
    const int32_t n = g.n;
    std::vector<std::vector<int32_t>> edges(static_cast<size_t>(n));
    std::vector<uint8_t> unary(static_cast<size_t>(n), 0);
    for (const auto& p : g.prods) {
        if (p.rhs.empty())
            unary[size_t(p.head)] = 1;
        else
            edges[size_t(p.head)].push_back(p.rhs.back());
    }
    g.adj.assign(size_t(n) * size_t(n), 0);
    std::vector<int32_t> queue;
    std::vector<uint8_t> seen;
    for (const auto& p : g.prods) {
        for (size_t i = 1; i < p.rhs.size(); ++i) {
            const int32_t z = p.rhs[i];
            seen.assign(size_t(n), 0);
            queue.clear();
            queue.push_back(p.rhs[i - 1]);
            seen[size_t(p.rhs[i - 1])] = 1;
            for (size_t q = 0; q < queue.size(); ++q) {
                const int32_t x = queue[q];
                if (unary[size_t(x)]) g.adj[size_t(x) * size_t(n) + size_t(z)] = 1;
                for (int32_t y : edges[size_t(x)])
                    if (!seen[size_t(y)]) {
                        seen[size_t(y)] = 1;
                        queue.push_back(y);
                    }
            }
        }
    }
}

// Algorithm 1 as a depth-first enumeration with explicit stacks. `prev` is the symbol popped last (-1: none yet).
struct Displacer {
    const cfgzip_grammar& g;
    const uint8_t* t;
    int32_t len;
    int64_t max_pairs;
    std::set<Pair> out;
    bool overflow = false;
    Stack s_in, s_out;  // s_out: top at the back

    void run(int32_t pos, int32_t prev) {
        if (overflow) return;
        if (pos == len) {
            Pair p(s_in, Stack(s_out.rbegin(), s_out.rend()));
            out.insert(std::move(p));
            if (int64_t(out.size()) > max_pairs) overflow = true;
            return;
        }
        const auto& cands = g.by_term[t[pos]];
        if (s_out.empty()) {  // stack backtrack: the next symbol of the input stack is guessed
            for (int32_t pi : cands) {
                const auto& p = g.prods[size_t(pi)];
                if (prev >= 0 && !g.adj[size_t(prev) * size_t(g.n) + size_t(p.head)]) continue;
                s_in.push_back(p.head);
                for (auto it = p.rhs.rbegin(); it != p.rhs.rend(); ++it) s_out.push_back(*it);
                run(pos + 1, p.head);
                s_out.resize(s_out.size() - p.rhs.size());
                s_in.pop_back();
            }
        } else {
            const int32_t top = s_out.back();
            for (int32_t pi : cands) {
                const auto& p = g.prods[size_t(pi)];
                if (p.head != top) continue;
                s_out.pop_back();
                for (auto it = p.rhs.rbegin(); it != p.rhs.rend(); ++it) s_out.push_back(*it);
                run(pos + 1, top);
                s_out.resize(s_out.size() - p.rhs.size());
                s_out.push_back(top);
            }
        }
    }
};

}  // namespace

extern "C" {

int cfgzip_grammar_create(int32_t n_nonterminals, int32_t start, const int32_t* prod_head, const uint8_t* prod_terminal,
                          const int32_t* prod_rhs_off, const int32_t* prod_rhs, int32_t n_prod, cfgzip_grammar** out) {
    if (!out) return CFGZIP_E_ARG;
    *out = nullptr;
    if (n_nonterminals <= 0 || start < 0 || start >= n_nonterminals || n_prod < 0) return CFGZIP_E_ARG;
    if (n_prod > 0 && (!prod_head || !prod_terminal || !prod_rhs_off)) return CFGZIP_E_ARG;
    cfgzip_grammar* g = new (std::nothrow) cfgzip_grammar();
    if (!g) return CFGZIP_E_NOMEM;
    g->n = n_nonterminals;
    g->start = start;
    g->by_term.resize(256);
    for (int32_t i = 0; i < n_prod; ++i) {
        const int32_t lo = prod_rhs_off[i], hi = prod_rhs_off[i + 1];
        bool ok = prod_head[i] >= 0 && prod_head[i] < n_nonterminals && lo >= 0 && hi >= lo && (hi == lo || prod_rhs);
        cfgzip_grammar::Prod p{prod_head[i], prod_terminal[i], {}};
        for (int32_t j = lo; ok && j < hi; ++j) {
            ok = prod_rhs[j] >= 0 && prod_rhs[j] < n_nonterminals;
            p.rhs.push_back(prod_rhs[j]);
        }
        if (!ok) {
            delete g;
            return CFGZIP_E_RANGE;
        }
        g->by_term[p.term].push_back(int32_t(g->prods.size()));
        g->prods.push_back(std::move(p));
    }
    build_adjacency(*g);
    *out = g;
    return CFGZIP_OK;
}

int cfgzip_grammar_destroy(cfgzip_grammar* g) {
    if (!g) return CFGZIP_E_ARG;
    delete g;
    return CFGZIP_OK;
}

int cfgzip_grammar_adjacency(const cfgzip_grammar* g, uint8_t* adjacency) {
    if (!g || !adjacency) return CFGZIP_E_ARG;
    std::memcpy(adjacency, g->adj.data(), g->adj.size());
    return CFGZIP_OK;
}

int cfgzip_displacement_signatures(const cfgzip_grammar* g, const uint8_t* token_bytes, const int64_t* token_off, int32_t V,
                                   int32_t row_words, int32_t* signatures, int32_t* signature_words, int64_t max_pairs) {
    if (!g || !token_off || V < 0 || row_words < 1 || !signatures || max_pairs < 1) return CFGZIP_E_ARG;
    if (V > 0 && !token_bytes && token_off[V] > token_off[0]) return CFGZIP_E_ARG;
    int rc = CFGZIP_OK;
    std::vector<int32_t> flat;
    for (int32_t i = 0; i < V; ++i) {
        const int64_t lo = token_off[i], hi = token_off[i + 1];
        if (hi < lo || hi - lo > 0x7FFFFFFF) return CFGZIP_E_ARG;
        Displacer d{*g, token_bytes + lo, int32_t(hi - lo), max_pairs};
        d.run(0, -1);  // (an empty token moves no stack: its only pair is (empty, empty))
        int32_t* row = signatures + int64_t(i) * row_words;
        std::fill(row, row + row_words, 0);
        if (d.overflow) {
            if (signature_words) signature_words[i] = -1;
            rc = CFGZIP_E_RANGE;
            continue;
        }
        // canonical sequence: the pairs in lexicographic order (std::set of pairs of vectors), each as
        // len(sigma_i), sigma_i, len(sigma_o), sigma_o
        flat.clear();
        for (const Pair& p : d.out) {
            flat.push_back(int32_t(p.first.size()));
            flat.insert(flat.end(), p.first.begin(), p.first.end());
            flat.push_back(int32_t(p.second.size()));
            flat.insert(flat.end(), p.second.begin(), p.second.end());
        }
        if (signature_words) signature_words[i] = int32_t(flat.size());
        if (int64_t(flat.size()) + 1 > row_words) {
            rc = CFGZIP_E_RANGE;
            continue;
        }
        row[0] = int32_t(flat.size());
        std::copy(flat.begin(), flat.end(), row + 1);
    }
    return rc;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------------------
// Grouping on the GPU. Tokens whose signature rows are equal word for word form a class. An open-addressing table
// keyed by the row CONTENT (a hash only picks the first slot; a slot is shared only after the rows compared equal)
// gives every token the slot of its class; the lowest token id of a slot names the class, classes are numbered in
// the order of those lowest ids (a prefix sum over "I am the lowest id of my class" flags), the representative is
// the member with the smallest (byte length, id), and the class lists are filled in ascending token id.
// ---------------------------------------------------------------------------------------------------------------
namespace {

constexpr int kScanThreads = 1024;

__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__global__ void k_group_insert(const int32_t* __restrict__ sig, int W, const int32_t* __restrict__ len, int V, int32_t* owner,
                               unsigned table_mask, int32_t* slot_of, int32_t* min_id, unsigned long long* rep_key) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= V) return;
    const int32_t* row = sig + int64_t(t) * W;
    unsigned long long h = 0x243F6A8885A308D3ull;
    for (int w = 0; w < W; ++w) h = mix64(h ^ static_cast<unsigned>(row[w]));
    unsigned slot = unsigned(h) & table_mask;
    for (unsigned probe = 0; probe <= table_mask; ++probe) {  // the table has at least 2 V slots: a free one always turns up
        int32_t o = atomicCAS(owner + slot, -1, t);
        bool same = o == -1 || o == t;
        if (!same) {
            const int32_t* other = sig + int64_t(o) * W;
            same = true;
            for (int w = 0; w < W && same; ++w) same = other[w] == row[w];
        }
        if (same) break;
        slot = (slot + 1) & table_mask;
    }
    slot_of[t] = int32_t(slot);
    atomicMin(min_id + slot, t);
    atomicMin(rep_key + slot, (static_cast<unsigned long long>(unsigned(len[t])) << 32) | unsigned(t));
}

// flag[t] = 1 when t is the lowest token id of its class
__global__ void k_group_flags(const int32_t* slot_of, const int32_t* min_id, int V, int32_t* flag) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < V) flag[t] = min_id[slot_of[t]] == t ? 1 : 0;
}

// Exclusive prefix sum of n integers in place, by one block; the total goes to *total (if not null) and to data[n].
__global__ void __launch_bounds__(kScanThreads) k_exclusive_scan(int32_t* data, int n, int32_t* total) {
    __shared__ int s_warp[kScanThreads / 32];
    __shared__ int s_carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int base = 0; base < n; base += kScanThreads) {
        const int i = base + tid;
        const int v = i < n ? data[i] : 0;
        int inc = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(0xFFFFFFFFu, inc, d);
            if (lane >= d) inc += up;
        }
        if (lane == 31) s_warp[warp] = inc;
        __syncthreads();
        int before = s_carry;
        for (int w = 0; w < warp; ++w) before += s_warp[w];
        if (i < n) data[i] = before + inc - v;
        __syncthreads();
        if (tid == kScanThreads - 1) s_carry = before + inc;
        __syncthreads();
    }
    if (tid == 0) {
        data[n] = s_carry;
        if (total) *total = s_carry;
    }
}

__global__ void k_group_assign(const int32_t* slot_of, const int32_t* min_id, const unsigned long long* rep_key,
                               const int32_t* class_of_first, int V, int32_t* c, int32_t* r, int32_t* count) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= V) return;
    const int slot = slot_of[t];
    const int first = min_id[slot];
    const int k = class_of_first[first];
    c[t] = k;
    atomicAdd(count + k, 1);
    if (first == t) r[k] = int32_t(rep_key[slot] & 0xFFFFFFFFull);
}

// Class lists in ascending token id: one warp walks the tokens in order, 32 at a time; lanes of the same class share
// one cursor and take consecutive places in lane order. The cursors (class offsets to start with) sit in shared
// memory when there are few enough classes, which takes the round trip to L2 out of every step of the walk.
constexpr int kListCursorsShared = 48 * 1024 / 4;

__global__ void __launch_bounds__(32) k_group_lists(const int32_t* c, int V, const int32_t* n_classes, int32_t* cursor,
                                                    int32_t* tok) {
    __shared__ int32_t s_cursor[kListCursorsShared];
    const int lane = threadIdx.x;
    const int K = *n_classes;
    const bool shared = K <= kListCursorsShared;
    int32_t* cur = shared ? s_cursor : cursor;
    if (shared) {
        for (int k = lane; k < K; k += 32) s_cursor[k] = cursor[k];
        __syncwarp();
    }
    int k_next = lane < V ? c[lane] : 0;  // the class of this lane's next token is fetched one round ahead
    for (int base = 0; base < V; base += 32) {
        const int t = base + lane;
        const bool have = t < V;
        const int k = have ? k_next : -1 - lane;  // lanes without a token match nobody
        if (t + 32 < V) k_next = c[t + 32];
        const unsigned peers = __match_any_sync(0xFFFFFFFFu, k);
        const int rank = __popc(peers & ((1u << lane) - 1u));
        const int leader = __ffs(peers) - 1;
        int at = 0;
        if (have && lane == leader) at = atomicAdd(cur + k, __popc(peers));
        at = __shfl_sync(0xFFFFFFFFu, at, leader);
        if (have) tok[at + rank] = t;
        __syncwarp();
    }
}

inline unsigned blocks_for(int n, int threads) { return unsigned((n + threads - 1) / threads); }

}  // namespace

extern "C" int cfgzip_group_tokens(const int32_t* signatures, int32_t row_words, const int32_t* token_len, int32_t V,
                                   int32_t* token_to_class, int32_t* class_to_rep, int32_t* n_classes, int32_t* class_off,
                                   int32_t* class_tok, void* stream) {
    if (V < 0 || row_words < 1) return CFGZIP_E_ARG;
    if (V == 0) return CFGZIP_OK;
    if (!signatures || !token_len || !token_to_class || !class_to_rep || !n_classes) return CFGZIP_E_ARG;
    if ((class_off == nullptr) != (class_tok == nullptr)) return CFGZIP_E_ARG;
    if (V > (1 << 28)) return CFGZIP_E_RANGE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned table = 1;
    while (table < 2u * unsigned(V)) table <<= 1;
    // scratch: owner, min_id [table]; rep_key [table]; slot_of, flag (+1), count (+1), cursor [V]
    const size_t n_i32 = size_t(table) * 2 + size_t(V) * 4 + 2;
    int32_t* i32 = nullptr;
    unsigned long long* rep_key = nullptr;
    if (cudaMalloc(&i32, n_i32 * sizeof(int32_t)) != cudaSuccess || cudaMalloc(&rep_key, size_t(table) * 8) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(i32);
        return CFGZIP_E_NOMEM;
    }
    int32_t* owner = i32;
    int32_t* min_id = owner + table;
    int32_t* slot_of = min_id + table;
    int32_t* flag = slot_of + V;       // V + 1 entries
    int32_t* count = flag + V + 1;     // V + 1 entries
    int32_t* cursor = count + V + 1;   // V entries
    bool ok = cudaMemsetAsync(owner, 0xFF, size_t(table) * 4, st) == cudaSuccess &&          // -1
              cudaMemsetAsync(min_id, 0x7F, size_t(table) * 4, st) == cudaSuccess &&         // a large positive id
              cudaMemsetAsync(rep_key, 0xFF, size_t(table) * 8, st) == cudaSuccess &&
              cudaMemsetAsync(count, 0, size_t(V + 1) * 4, st) == cudaSuccess;
    if (ok) {
        const int T = 256;
        k_group_insert<<<blocks_for(V, T), T, 0, st>>>(signatures, row_words, token_len, V, owner, table - 1, slot_of, min_id,
                                                       rep_key);
        k_group_flags<<<blocks_for(V, T), T, 0, st>>>(slot_of, min_id, V, flag);
        k_exclusive_scan<<<1, kScanThreads, 0, st>>>(flag, V, n_classes);
        k_group_assign<<<blocks_for(V, T), T, 0, st>>>(slot_of, min_id, rep_key, flag, V, token_to_class, class_to_rep, count);
        if (class_off) {
            // class sizes -> offsets (the scan also writes the total V behind the last class that exists: entries past
            // n_classes all read V), then the lists
            k_exclusive_scan<<<1, kScanThreads, 0, st>>>(count, V, nullptr);
            ok = cudaMemcpyAsync(class_off, count, size_t(V + 1) * 4, cudaMemcpyDeviceToDevice, st) == cudaSuccess &&
                 cudaMemcpyAsync(cursor, count, size_t(V) * 4, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
            if (ok) k_group_lists<<<1, 32, 0, st>>>(token_to_class, V, n_classes, cursor, class_tok);
        }
        ok = ok && cudaGetLastError() == cudaSuccess;
    }
    ok = (cudaStreamSynchronize(st) == cudaSuccess) && ok;  // the scratch is released below
    cudaFree(i32);
    cudaFree(rep_key);
    if (!ok) {
        cudaGetLastError();
        return CFGZIP_E_CUDA;
    }
    return CFGZIP_OK;
}
