// Device-side building blocks shared by the kernels: partition descriptors, the
// (max, sum-exp, position) partial state and its merge, bit-matrix transposes,
// and 16-byte "octet" (8 tokens) loads and stores.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace cfgzip {

constexpr int kGroupRows = 32;        // rows that share one bit-sliced class table
constexpr int kBatchRows = 8;         // rows a warp streams together
constexpr int kNoPos = 0x7FFFFFFF;    // "no allowed token seen"
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRefFloor = -1.7e38f; // lowest reference used for exp(z - ref)

enum : int { kF32 = 0, kBF16 = 1 };

// One loaded partition, as the kernels see it (all pointers are device memory).
struct PartDev {
    const uint16_t* c16;   // token -> class, padded to 32*VW entries with the value K; null when K > 65535
    const int32_t* c32;    // token -> class, V entries
    const int32_t* r;      // class -> representative token, K entries
    const int32_t* off;    // class -> start in tok, K+1 entries
    const int32_t* tok;    // tokens grouped by class, ascending inside a class
    const int32_t* trep;   // token -> representative of its class, r[c[t]], V entries (one load instead of two in a chain)
    int32_t K;
    int32_t KW;
    int32_t V;
    int32_t live;          // 0 when the slot is free
};

// Per-row reduction state. m: largest allowed logit seen (-inf if none or all -inf);
// s: sum of exp(z - max(m, kRefFloor)) over allowed logits; pos: position (octet or
// token index, ascending with the token id) of the first occurrence of m.
struct Partial {
    float m;
    float s;
    int pos;
    int pad;
};

__device__ __forceinline__ Partial partial_empty() { return Partial{-INFINITY, 0.f, kNoPos, 0}; }

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Total order used at every level: larger value wins; equal values: lower position.
// The sums are brought to the larger reference before they are added. `scale` is log2(e) / T:
// the sums are of exp(z / T) (T = 1 everywhere except in a sampling step).
__device__ __forceinline__ void partial_merge(float& m, float& s, int& pos, float m2, float s2, int pos2,
                                              float scale = kLog2e) {
    const float r1 = fmaxf(m, kRefFloor), r2 = fmaxf(m2, kRefFloor);
    const float d = r1 - r2;
    const float e = ex2f(-fabsf(d) * scale);
    s = d >= 0.f ? fmaf(s2, e, s) : fmaf(s, e, s2);
    const bool take2 = (m2 > m) || (m2 == m && pos2 < pos);
    pos = take2 ? pos2 : pos;
    m = fmaxf(m, m2);
}

// Butterfly all-reduce of one row's state over the 32 lanes of a warp.
__device__ __forceinline__ void partial_warp_allreduce(float& m, float& s, int& pos, float scale = kLog2e) {
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        const float m2 = __shfl_xor_sync(0xFFFFFFFFu, m, d);
        const float s2 = __shfl_xor_sync(0xFFFFFFFFu, s, d);
        const int p2 = __shfl_xor_sync(0xFFFFFFFFu, pos, d);
        partial_merge(m, s, pos, m2, s2, p2, scale);
    }
}

// 32x32 bit-matrix transpose across a warp: on entry lane r holds row r (bit j = column
// j); on return lane j holds column j (bit r = row r). Five block-swap stages.
__device__ __forceinline__ uint32_t warp_transpose32(uint32_t x, int lane) {
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        // low mask of each 2d-wide bit block: d=16 -> 0x0000FFFF, 8 -> 0x00FF00FF, ...
        const uint32_t lo = 0xFFFFFFFFu / ((1u << d) + 1u);
        const uint32_t y = __shfl_xor_sync(0xFFFFFFFFu, x, d);
        x = (lane & d) ? ((y >> d) & lo) | (x & ~lo) : (x & lo) | ((y & lo) << d);
    }
    return x;
}

// 8x8 bit-matrix transpose held in two registers. On entry byte j of (lo, hi) -- lo holds
// j = 0..3, hi holds j = 4..7 -- is row j, bit i of that byte is column i. On return byte i
// is column i with bit j = old row j.
__host__ __device__ __forceinline__ void transpose8x8(uint32_t& lo, uint32_t& hi) {
    uint32_t t;
    // swap the off-diagonal 4x4 blocks (rows 0-3 / cols 4-7 with rows 4-7 / cols 0-3)
    t = ((lo >> 4) ^ hi) & 0x0F0F0F0Fu;
    hi ^= t;
    lo ^= t << 4;
    // 2x2 blocks inside each 4x4: rows j and j+2 are 16 bits apart inside one register
    t = (lo ^ (lo >> 14)) & 0x0000CCCCu;
    lo ^= t ^ (t << 14);
    t = (hi ^ (hi >> 14)) & 0x0000CCCCu;
    hi ^= t ^ (t << 14);
    // single bits inside each 2x2: rows j and j+1 are 8 bits apart
    t = (lo ^ (lo >> 7)) & 0x00AA00AAu;
    lo ^= t ^ (t << 7);
    t = (hi ^ (hi >> 7)) & 0x00AA00AAu;
    hi ^= t ^ (t << 7);
}

// Spread the 4 bits of a nibble to the top bit of the 4 bytes of a word (bit j -> bit 8j+7).
__device__ __forceinline__ uint32_t nibble_to_byte_msbs(uint32_t nib) { return nib * 0x10204080u; }

// PTX byte permute in its default mode: selector nibble n picks byte (n & 7) of {b, a};
// with bit 3 of the nibble set, the top bit of that byte is replicated over the result byte.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Streaming 16-byte accesses for the logits (read once, written once).
__device__ __forceinline__ uint4 ld_stream16(const void* p) { return __ldcs(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ void st_stream16(void* p, uint4 v) { __stcs(reinterpret_cast<uint4*>(p), v); }
// One 32-byte store (p 32-byte aligned). Two 16-byte stores per lane would leave every 32-byte sector half
// written by each of the two instructions of a warp; written whole, a write-only pass runs about twice as fast.
__device__ __forceinline__ void st_stream32(void* p, uint4 lo, uint4 hi) {
    asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w),
                 "r"(hi.x), "r"(hi.y), "r"(hi.z), "r"(hi.w)
                 : "memory");
}

// Logit element access by dtype (scalar, for ragged tails and unaligned buffers).
template <int DT>
__device__ __forceinline__ float load_elem(const void* base, int64_t idx) {
    if (DT == kBF16) return __uint_as_float(uint32_t(reinterpret_cast<const uint16_t*>(base)[idx]) << 16);
    return reinterpret_cast<const float*>(base)[idx];
}
template <int DT>
__device__ __forceinline__ void store_neg_inf(void* base, int64_t idx) {
    if (DT == kBF16)
        reinterpret_cast<uint16_t*>(base)[idx] = 0xFF80u;
    else
        reinterpret_cast<uint32_t*>(base)[idx] = 0xFF800000u;
}

// Eight consecutive logits of one row ("octet"), masked by the 8 allow bits in `byte`:
// the masked values land in f[0..7] and the masked bit patterns in the registers that are
// stored back. bf16: one 16-byte vector; f32: two.
template <int DT>
struct Octet;

template <>
struct Octet<kBF16> {
    uint4 v;
    __device__ __forceinline__ void load(const void* row_base, int o) {
        v = ld_stream16(reinterpret_cast<const uint16_t*>(row_base) + 8 * int64_t(o));
    }
    __device__ __forceinline__ void load_shared(const char* stage_row, int lane) {
        v = *reinterpret_cast<const uint4*>(stage_row + lane * 16);
    }
    __device__ __forceinline__ void load_shared_at(const char* p) { v = *reinterpret_cast<const uint4*>(p); }
    __device__ __forceinline__ void store(void* row_base, int o) const {
        st_stream16(reinterpret_cast<uint16_t*>(row_base) + 8 * int64_t(o), v);
    }
    __device__ __forceinline__ void store_at(void* p) const { st_stream16(p, v); }
    __device__ __forceinline__ void store(void* row_base, int o, bool) const { store(row_base, o); }
    __device__ __forceinline__ void store_at(void* p, bool) const { store_at(p); }
    __device__ __forceinline__ void fill_neg_inf() { v = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u); }
    __device__ __forceinline__ uint4 raw() const { return v; }
    __device__ __forceinline__ void mask(uint32_t byte, float* f) {
        const uint32_t xl = nibble_to_byte_msbs(byte & 0xFu), xh = nibble_to_byte_msbs(byte >> 4);
        // replicate the top bit of byte 2p / 2p+1 over the low / high half-word
        const uint32_t m0 = prmt(xl, 0u, 0x9988), m1 = prmt(xl, 0u, 0xBBAA);
        const uint32_t m2 = prmt(xh, 0u, 0x9988), m3 = prmt(xh, 0u, 0xBBAA);
        const uint32_t ni = 0xFF80FF80u;
        v.x = (v.x & m0) | (ni & ~m0);
        v.y = (v.y & m1) | (ni & ~m1);
        v.z = (v.z & m2) | (ni & ~m2);
        v.w = (v.w & m3) | (ni & ~m3);
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
        f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
        f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
    }
};

template <>
struct Octet<kF32> {
    uint4 a, b;
    __device__ __forceinline__ void load(const void* row_base, int o) {
        const float* p = reinterpret_cast<const float*>(row_base) + 8 * int64_t(o);
        a = ld_stream16(p);
        b = ld_stream16(p + 4);
    }
    __device__ __forceinline__ void load_shared(const char* stage_row, int lane) {
        a = *reinterpret_cast<const uint4*>(stage_row + lane * 32);
        b = *reinterpret_cast<const uint4*>(stage_row + lane * 32 + 16);
    }
    __device__ __forceinline__ void load_shared_at(const char* p) {
        a = *reinterpret_cast<const uint4*>(p);
        b = *reinterpret_cast<const uint4*>(p + 16);
    }
    __device__ __forceinline__ void store(void* row_base, int o) const {
        float* p = reinterpret_cast<float*>(row_base) + 8 * int64_t(o);
        st_stream16(p, a);
        st_stream16(p + 4, b);
    }
    __device__ __forceinline__ void store_at(void* p) const {
        st_stream16(p, a);
        st_stream16(reinterpret_cast<char*>(p) + 16, b);
    }
    // wide: the octet's address is 32-byte aligned (the caller knows it for the whole buffer)
    __device__ __forceinline__ void store_at(void* p, bool wide) const {
        if (wide) st_stream32(p, a, b); else store_at(p);
    }
    __device__ __forceinline__ void store(void* row_base, int o, bool wide) const {
        store_at(reinterpret_cast<float*>(row_base) + 8 * int64_t(o), wide);
    }
    __device__ __forceinline__ void fill_neg_inf() {
        a = make_uint4(0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u);
        b = a;
    }
    __device__ __forceinline__ uint4 raw() const { return a; }  // only called for bf16 (two octets per lane)
    __device__ __forceinline__ void mask(uint32_t byte, float* f) {
        const uint32_t xl = nibble_to_byte_msbs(byte & 0xFu), xh = nibble_to_byte_msbs(byte >> 4);
        const uint32_t ni = 0xFF800000u;
        uint32_t m;
        m = prmt(xl, 0u, 0x8888); a.x = (a.x & m) | (ni & ~m);
        m = prmt(xl, 0u, 0x9999); a.y = (a.y & m) | (ni & ~m);
        m = prmt(xl, 0u, 0xAAAA); a.z = (a.z & m) | (ni & ~m);
        m = prmt(xl, 0u, 0xBBBB); a.w = (a.w & m) | (ni & ~m);
        m = prmt(xh, 0u, 0x8888); b.x = (b.x & m) | (ni & ~m);
        m = prmt(xh, 0u, 0x9999); b.y = (b.y & m) | (ni & ~m);
        m = prmt(xh, 0u, 0xAAAA); b.z = (b.z & m) | (ni & ~m);
        m = prmt(xh, 0u, 0xBBBB); b.w = (b.w & m) | (ni & ~m);
        f[0] = __uint_as_float(a.x); f[1] = __uint_as_float(a.y);
        f[2] = __uint_as_float(a.z); f[3] = __uint_as_float(a.w);
        f[4] = __uint_as_float(b.x); f[5] = __uint_as_float(b.y);
        f[6] = __uint_as_float(b.z); f[7] = __uint_as_float(b.w);
    }
};

__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Packed pairs of floats (sm_100 has two-wide fp32 multiply-add and add).
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long p;
    asm("mov.b64 %0, {%1, %2};" : "=l"(p) : "f"(lo), "f"(hi));
    return p;
}
__device__ __forceinline__ void unpack2(unsigned long long p, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// One byte to global memory. Written as an explicit global store so that the compiler does not
// have to order it against shared-memory accesses (a pointer that comes out of inline assembly is
// generic to it); nothing in a kernel reads these bytes back.
__device__ __forceinline__ void st_global_u8(void* p, uint32_t v) {
    asm volatile("st.global.u8 [%0], %1;" ::"l"(p), "r"(v));
}

__device__ __forceinline__ void st_global_u16(void* p, uint32_t v) {
    asm volatile("st.global.u16 [%0], %1;" ::"l"(p), "h"(static_cast<unsigned short>(v)));
}

// base + i * stride with a 32-bit stride in one wide multiply-add
__device__ __forceinline__ char* ptr_mad(char* base, uint32_t i, uint32_t stride) {
    unsigned long long r;
    asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(r) : "r"(i), "r"(stride), "l"(reinterpret_cast<unsigned long long>(base)));
    return reinterpret_cast<char*>(r);
}

// Running state of one row inside one thread. The sum is kept relative to a reference that
// only moves when a value overtakes it by more than kRefSlack (so the common case is one
// fused multiply-add and one ex2 per logit): s = sum 2^(z*scale + nrl), nrl = -(ref*scale), with
// scale = log2(e) / T. pos is the position (octet index) of the first octet whose maximum is the
// row maximum m.
constexpr float kRefSlack = 57.7f;  // in powers of two: 40 nats
struct RowAcc {
    float m, s, nrl;
    int pos;
    __device__ __forceinline__ void init() {
        m = -INFINITY;
        s = 0.f;
        nrl = -(kRefFloor * kLog2e);
        pos = kNoPos;
    }
    // N = 8 or 16 consecutive logits of the row (masked ones are -inf), `position` the index of their first octet.
    template <int N>
    __device__ __forceinline__ void add_values(const float* f, int position, float scale = kLog2e) {
        float vmax = fmax3(fmax3(f[0], f[1], f[2]), fmax3(f[3], f[4], f[5]), fmaxf(f[6], f[7]));
        if (N == 16)
            vmax = fmaxf(vmax, fmax3(fmax3(f[8], f[9], f[10]), fmax3(f[11], f[12], f[13]), fmaxf(f[14], f[15])));
        pos = vmax > m ? position : pos;
        m = fmaxf(m, vmax);
        if (fmaf(vmax, scale, nrl) > kRefSlack) {  // rare: move the reference up to vmax
            const float n2 = -(vmax * scale);
            s *= ex2f(n2 - nrl);
            nrl = n2;
        }
        const unsigned long long l2 = pack2(scale, scale), n2p = pack2(nrl, nrl);
        unsigned long long e2[N / 2];
#pragma unroll
        for (int j = 0; j < N; j += 2) {
            float t0, t1;
            unpack2(fma2(pack2(f[j], f[j + 1]), l2, n2p), t0, t1);
            e2[j / 2] = pack2(ex2f(t0), ex2f(t1));
        }
#pragma unroll
        for (int w = N / 4; w >= 1; w >>= 1)
#pragma unroll
            for (int j = 0; j < w; ++j) e2[j] = add2(e2[j], e2[j + w]);
        float a0, a1;
        unpack2(e2[0], a0, a1);
        s += a0 + a1;
    }
    __device__ __forceinline__ void add_octet(const float (&f)[8], int position, float scale = kLog2e) {
        add_values<8>(f, position, scale);
    }
    // Bring the sum to the convention of Partial: relative to max(m, kRefFloor).
    __device__ __forceinline__ Partial to_partial(float scale = kLog2e) const {
        // nothing finite seen: the reference never moved off the floor and the sum is empty
        if (!(m > kRefFloor)) return Partial{m, 0.f, pos, 0};
        return Partial{m, s * ex2f(-fmaf(m, scale, nrl)), pos, 0};
    }
};

// ---- mbarrier + bulk asynchronous copy (global -> shared) wrappers, CTA scope ----------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// One bounded attempt: returns true once the phase with the given parity has completed.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(2000u)
        : "memory");
    return ok != 0;
}
// Bounded wait (about half a second at most); false means the copy never arrived.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (int it = 0; it < 250000; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// Tiled 2-D copy through a tensor map: box of (x .. x+boxDim0) elements by (y .. y+boxDim1) rows.
// x times the element size must be a multiple of 16 bytes; out-of-range parts are zero-filled.
__device__ __forceinline__ void tma_g2s_2d(void* dst_smem, const void* tensor_map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_u32(dst_smem)),
        "l"(tensor_map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
// The same box into the L2 only (a hint: nothing is delivered, no barrier involved).
__device__ __forceinline__ void tma_prefetch_2d(const void* tensor_map, int x, int y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(tensor_map), "r"(x), "r"(y) : "memory");
}
// size and address multiples of 16 bytes; into the L2 only
__device__ __forceinline__ void bulk_prefetch(const void* src_gmem, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src_gmem), "r"(bytes) : "memory");
}
// size and both addresses are multiples of 16 bytes
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

}  // namespace cfgzip
