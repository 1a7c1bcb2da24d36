// Device side of the library: upload of a built format and the fused decode-multiply-accumulate
// kernels for HAC (Algorithm 1) and sHAC (Algorithm 2), for one input and for a batch
// (Algorithm 3), written for sm_100a.
//
// Work decomposition.  The offset index cuts every column into sub-segments of S symbols; 32
// consecutive sub-segments form a segment, the work unit of one warp.  A warp reads the 32
// sub-segment bit lengths, turns them into per-lane start bits with a shuffle scan, copies the
// segment's span of the stream into shared memory with 128-bit coalesced loads, and then every
// lane decodes its own sub-segment from shared memory with a table lookup per code word.  Partial
// dot products are combined with warp shuffles; columns that span several segments are finished
// by a small second kernel that adds the per-segment partials in a fixed order.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <utility>
#include <string>
#include <type_traits>

#include "hac_internal.h"

namespace hacb200 {

static thread_local std::string g_last_cuda_error;

static int cuda_fail(cudaError_t e, const char* what) {
    g_last_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
    return HAC_ERR_CUDA;
}
#define HAC_CUDA(call)                                              \
    do {                                                            \
        cudaError_t e_ = (call);                                    \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call);         \
    } while (0)

// ------------------------------------------------------------------------------------------------
// Kernel-side view of a format (device pointers and scalars), passed by value.
// ------------------------------------------------------------------------------------------------
struct DevFormat {
    const uint32_t* stream;
    const uint16_t* lut;
    const uint2* l1;
    const uint2* sub;
    const float* rank_value;
    const uint64_t* limit;
    const uint32_t* first_left;
    const uint32_t* rank_base;
    const uint64_t* seg_bit_off;
    const uint16_t* sub_bits;
    const uint32_t* seg_col;
    const uint32_t* seg_first;
    const void* ri;
    const uint32_t* cb;
    const void* unit_info;
    uint32_t n, m, units, G, S, k_eff, lut_bits, max_len, ri_bits, max_unit_chunks, max_sub_chunks, l1_bits, sub_bytes, items;
    // First-level table `l1`, l1_entries entries.  tab_kind 0: the prefix table (2^l1_bits entries).  1: the
    // magnitude table with xt_mant mantissa bits, rows xt_row0 .. 31 (the rows below belong to windows with more
    // leading ones than the longest code word has bits: xt_low, OR-ed into ~window, keeps the index out of them);
    // its unresolved cells go to the search over lengths (no sub-tables).
    uint32_t tab_kind, l1_entries, xt_mant, xt_row0, xt_low;
    // what is done to an output before it is stored (layer evaluation): + bias[j], then max(., 0)
    const float* epi_bias;
    uint32_t epi_relu;
};

// The value stored for output j: the product, plus the layer's bias, through its activation.  (A NaN stays a NaN.)
__device__ __forceinline__ float finish_output(const float* __restrict__ bias, uint32_t relu, float v, uint32_t j) {
    if (bias) v += __ldg(bias + j);
    if (relu && v < 0.0f) v = 0.0f;
    return v;
}
__device__ __forceinline__ float finish_output(const DevFormat& f, float v, uint32_t j) {
    return finish_output(f.epi_bias, f.epi_relu, v, j);
}


// ------------------------------------------------------------------------------------------------
// All shared memory is one dynamic array; tables and staging areas are addressed by 32-bit byte
// offsets into it, which keeps address arithmetic in 32 bits and lets the compiler schedule the
// loads freely between the warp- and block-level barriers.
// ------------------------------------------------------------------------------------------------
extern __shared__ __align__(16) unsigned char smem[];

__device__ __forceinline__ uint32_t smem_off(const void* p) {
    return (uint32_t)(reinterpret_cast<const unsigned char*>(p) - smem);
}
__device__ __forceinline__ uint32_t lds32(uint32_t off) { return *reinterpret_cast<const uint32_t*>(smem + off); }
__device__ __forceinline__ uint32_t lds16(uint32_t off) { return *reinterpret_cast<const uint16_t*>(smem + off); }
__device__ __forceinline__ float ldsf(uint32_t off) { return *reinterpret_cast<const float*>(smem + off); }
__device__ __forceinline__ uint2 lds64(uint32_t off) { return *reinterpret_cast<const uint2*>(smem + off); }

__host__ __device__ inline size_t align16(size_t x) { return (x + 15) & ~(size_t)15; }

// How a kernel lays out its decoding tables in shared memory (replication chosen by the host).
//   level 1: the format's 2^l1_bits entries {value bits, length}, 8 bytes each, stored `repl` times
//            interleaved (entry i of replica r at index i*repl + r) so that lanes r, r+repl, .. read
//            disjoint banks.  An entry with the top bit of the second word set stands for a prefix
//            shared by longer code words: {byte offset of a sub-table, 0x80000000 | b}.
//   level 2: the sub-tables, one copy, indexed by the next b bits: {value bits, length}, or {0, 0}
//            for code words longer still, which are found by a search over lengths in global memory.
struct TablePlan {
    uint32_t repl_log2;
    uint32_t zero_len;    // HAC zero-run table in use: code length of the zero symbol
    uint32_t x_bulk;      // sHAC: x is contiguous and 16-byte aligned, so it is brought in by one bulk async copy
    uint32_t prefetch;    // HAC rows kernel: ask for the block's share of the stream into L2 at the start
};

__host__ __device__ inline size_t plan_smem_bytes(uint32_t l1_entries, uint32_t repl_log2, uint32_t sub_bytes) {
    return (((size_t)8 * l1_entries) << repl_log2) + align16(sub_bytes);
}

// Per-thread handle on the staged tables (shared-space addresses) and the global fallbacks.
struct Decoder {
    uint32_t l1_lane, l1_mul, l1_shift, l1_bits, sub;
    uint32_t bias;        // magnitude table: raw index of the first entry kept (subtracted from the raw index); else 0
    uint32_t xt_low;      // magnitude table: low bits OR-ed into ~window before the conversion
};

// TF32 split of a shared value for the tensor-core kernel, packed with the code length:
//   .y = hi | length   (hi = the value rounded to TF32: its low 13 bits are zero, the length, at most 32, sits in the low 6)
//   .x = lo            (the remainder value - hi, rounded to TF32)
// An entry that stands for a prefix of longer code words becomes {byte offset of the sub-table,
// kSplitLong | b}; a sub-table slot of a code word longer still stays {0, 0}.
constexpr uint32_t kSplitLong = 0x1000u;
__device__ __forceinline__ uint32_t round_tf32(float v) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ uint2 split_entry(uint2 e) {
    if ((int32_t)e.y < 0) return make_uint2(e.x, kSplitLong | (e.y & 31u));
    if (e.y == 0) return make_uint2(0u, 0u);
    const float v = __uint_as_float(e.x);
    const uint32_t hi = round_tf32(v) & 0xffffe000u;
    const uint32_t lo = round_tf32(v - __uint_as_float(hi)) & 0xffffe000u;
    return make_uint2(lo, hi | e.y);
}

// Builds the tables in shared memory (whole block takes part) and advances `p` past them.  With
// kSplit the entries are stored in the split form above.
template <bool kSplit = false>
__device__ __forceinline__ Decoder stage_decoder(const DevFormat& f, const TablePlan& tp, unsigned char*& p) {
    Decoder d;
    const uint32_t repl = 1u << tp.repl_log2;
    uint2* l1 = reinterpret_cast<uint2*>(p);
    p += ((size_t)8 * f.l1_entries) << tp.repl_log2;
    uint2* sub = reinterpret_cast<uint2*>(p);
    p += align16(f.sub_bytes);
    // Each thread loads one entry; the warp then writes its 32 entries' replicas slot by slot, the
    // value for a slot fetched from the lane that holds it, so that consecutive lanes write
    // consecutive 8-byte slots (no bank conflicts) and every entry is read from memory once.
    const uint32_t lane_ = threadIdx.x & 31u;
    // all loads of the first pass are issued before any of them is used, so that the block pays
    // one trip to memory for its tables, not one per table
    constexpr int kSubAhead = 4;
    uint2 sub_v[kSubAhead];
    const uint32_t sub_entries = f.sub_bytes / 8;
#pragma unroll
    for (int k = 0; k < kSubAhead; ++k) {
        const uint32_t i = threadIdx.x + k * blockDim.x;
        sub_v[k] = i < sub_entries ? __ldg(f.sub + i) : make_uint2(0u, 0u);
        if (kSplit) sub_v[k] = split_entry(sub_v[k]);
    }
    for (uint32_t idx0 = threadIdx.x - lane_; idx0 < f.l1_entries; idx0 += blockDim.x) {
        const uint32_t idx = idx0 + lane_;
        uint2 v = make_uint2(0u, 0u);
        if (idx < f.l1_entries) v = __ldg(f.l1 + idx);
        if (kSplit) v = split_entry(v);
        uint2* dst = l1 + ((size_t)idx0 << tp.repl_log2);
        const uint32_t warp_slots = min(32u, f.l1_entries - idx0) << tp.repl_log2;
        for (uint32_t s0 = 0; s0 < warp_slots; s0 += 32) {
            const uint32_t src = (s0 + lane_) >> tp.repl_log2;
            uint2 w;
            w.x = __shfl_sync(0xffffffffu, v.x, src & 31u);
            w.y = __shfl_sync(0xffffffffu, v.y, src & 31u);
            if (s0 + lane_ < warp_slots) dst[s0 + lane_] = w;
        }
    }
#pragma unroll
    for (int k = 0; k < kSubAhead; ++k) {
        const uint32_t i = threadIdx.x + k * blockDim.x;
        if (i < sub_entries) sub[i] = sub_v[k];
    }
    for (uint32_t i = threadIdx.x + kSubAhead * blockDim.x; i < sub_entries; i += blockDim.x)
        sub[i] = kSplit ? split_entry(__ldg(f.sub + i)) : __ldg(f.sub + i);
    d.l1_lane = smem_off(l1) + ((threadIdx.x & (repl - 1)) << 3);
    d.l1_mul = 8u << tp.repl_log2;
    d.l1_shift = f.tab_kind ? 23 - f.xt_mant : 32 - f.l1_bits;
    d.bias = f.tab_kind ? (127u + f.xt_row0) << f.xt_mant : 0u;
    d.xt_low = f.xt_low;
    d.l1_bits = f.l1_bits;
    d.sub = smem_off(sub);
    return d;
}

// Per-lane bit reader over the staged span: a 64-bit window (hi, lo) that starts at a word
// boundary, `off` bits of it (< 32) already consumed, `next` = shared address of the word after lo.
struct BitReader {
    uint32_t hi, lo, off, next;
    __device__ __forceinline__ void init(uint32_t stage_addr, uint32_t bitpos) {
        const uint32_t a = stage_addr + ((bitpos >> 5) << 2);
        hi = lds32(a);
        lo = lds32(a + 4);
        off = bitpos & 31u;
        next = a + 8;
    }
    __device__ __forceinline__ uint32_t peek() const { return __funnelshift_l(lo, hi, off); }
    __device__ __forceinline__ void skip(uint32_t len) {
        off += len;
        if (off >= 32u) {
            hi = lo;
            lo = lds32(next);
            next += 4;
            off -= 32u;
        }
    }
};

// Code words longer than both table levels (rare): the format's full-width 16-bit table, then the
// search over lengths, all in global memory.
__device__ __noinline__ uint2 decode_long(uint32_t top, const uint16_t* __restrict__ lut, uint32_t lut_bits,
                                          const float* __restrict__ rank_value, const uint64_t* __restrict__ limit,
                                          const uint32_t* __restrict__ first_left,
                                          const uint32_t* __restrict__ rank_base, uint32_t max_len) {
    const uint32_t code = lut[top >> (32 - lut_bits)];
    uint32_t len = code & 15u, rank = code >> 4;       // lengths here are at most kLutBitsMax = 12
    if (len == 0) {
        len = max_len; rank = 0;
        for (uint32_t l = lut_bits + 1; l <= max_len; ++l) {
            if ((uint64_t)top < limit[l]) {
                len = l;
                rank = rank_base[l] + ((top - first_left[l]) >> (32 - l));
                break;
            }
        }
    }
    return make_uint2(__float_as_uint(rank_value[rank]), len);
}

// One code word -> the shared value it stands for.
template <bool kLong>
__device__ __forceinline__ float decode_value(BitReader& br, const Decoder& d, const DevFormat& f) {
    const uint32_t top = br.peek();
    uint2 e = lds64(d.l1_lane + (top >> d.l1_shift) * d.l1_mul);
    if (kLong) {
        if ((int32_t)e.y < 0) {
            const uint32_t q = (top << d.l1_bits) >> (32 - (e.y & 31u));
            e = lds64(d.sub + e.x + (q << 3));
            if (e.y == 0)
                e = decode_long(top, f.lut, f.lut_bits, f.rank_value, f.limit, f.first_left, f.rank_base, f.max_len);
        }
    }
    br.skip(e.y);
    return __uint_as_float(e.x);
}

// ------------------------------------------------------------------------------------------------
// Hand-scheduled decode step (PTX).  One step of one chain is split in two parts so that the parts
// of several chains can be interleaved in program order:
//   lookup : window -> level-1 entry                      (4 instructions)
//   consume: advance the window by the code length, refill it from the staged span when 32 bits
//            are used up, multiply-accumulate with x       (9 instructions)
// Shared memory is addressed by absolute 32-bit shared-space addresses here.
// ------------------------------------------------------------------------------------------------
struct FastReader {
    uint32_t hi, lo, off, next;          // next: shared address of the word after lo
};

__device__ __forceinline__ uint32_t shared_base() { return (uint32_t)__cvta_generic_to_shared(smem); }

__device__ __forceinline__ void fast_lookup(const FastReader& r, uint32_t l1_shift, uint32_t l1_mul, uint32_t l1_lane,
                                            uint32_t& top, uint32_t& val, uint32_t& len) {
    asm volatile(
        "{\n\t"
        ".reg .b32 i;\n\t"
        "shf.l.wrap.b32 %0, %3, %4, %5;\n\t"
        "shr.u32 i, %0, %6;\n\t"
        "mad.lo.u32 i, i, %7, %8;\n\t"
        "ld.shared.v2.u32 {%1, %2}, [i];\n\t"
        "}"
        : "=r"(top), "=r"(val), "=r"(len)
        : "r"(r.lo), "r"(r.hi), "r"(r.off), "r"(l1_shift), "r"(l1_mul), "r"(l1_lane)
        : "memory");
}

// The same lookup in the magnitude table: the index is the exponent and the leading mantissa bits of
// float(~window | 1), rounded toward zero (7 instructions).  `l1_lane` already has the index of exponent
// 127 taken off.
__device__ __forceinline__ void fast_lookup_xt(const FastReader& r, uint32_t l1_shift, uint32_t l1_mul, uint32_t l1_lane,
                                               uint32_t xt_low, uint32_t& top, uint32_t& val, uint32_t& len) {
    asm volatile(
        "{\n\t"
        ".reg .b32 i;\n\t"
        "shf.l.wrap.b32 %0, %3, %4, %5;\n\t"
        "lop3.b32 i, %0, %9, 0, 0xCF;\n\t"
        "cvt.rz.f32.u32 i, i;\n\t"
        "shr.u32 i, i, %6;\n\t"
        "mad.lo.u32 i, i, %7, %8;\n\t"
        "ld.shared.v2.u32 {%1, %2}, [i];\n\t"
        "}"
        : "=r"(top), "=r"(val), "=r"(len)
        : "r"(r.lo), "r"(r.hi), "r"(r.off), "r"(l1_shift), "r"(l1_mul), "r"(l1_lane), "r"(xt_low)
        : "memory");
}

template <int kTab>
__device__ __forceinline__ void table_lookup(const FastReader& r, uint32_t l1_shift, uint32_t l1_mul, uint32_t l1_lane,
                                             uint32_t xt_low, uint32_t& top, uint32_t& val, uint32_t& len) {
    if (kTab == 0) fast_lookup(r, l1_shift, l1_mul, l1_lane, top, val, len);
    else fast_lookup_xt(r, l1_shift, l1_mul, l1_lane, xt_low, top, val, len);
}

template <int kXOffset>
__device__ __forceinline__ void fast_consume(FastReader& r, uint32_t val, uint32_t len, uint32_t x_addr, float& acc) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        ".reg .f32 xv;\n\t"
        "ld.shared.f32 xv, [%7+%8];\n\t"
        "add.u32 %2, %2, %6;\n\t"
        "setp.ge.u32 p, %2, 32;\n\t"
        "@p mov.u32 %0, %1;\n\t"
        "@p ld.shared.u32 %1, [%3];\n\t"
        "@p add.u32 %3, %3, 4;\n\t"
        "and.b32 %2, %2, 31;\n\t"
        "fma.rn.f32 %4, xv, %5, %4;\n\t"
        "}"
        : "+r"(r.hi), "+r"(r.lo), "+r"(r.off), "+r"(r.next), "+f"(acc)
        : "f"(__uint_as_float(val)), "r"(len), "r"(x_addr), "n"(kXOffset)
        : "memory");
}

// The consume part alone (no multiply-accumulate): used where the decoded value goes to a tile.
__device__ __forceinline__ void fast_consume_value(FastReader& r, uint32_t len) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "add.u32 %2, %2, %4;\n\t"
        "setp.ge.u32 p, %2, 32;\n\t"
        "@p mov.u32 %0, %1;\n\t"
        "@p ld.shared.u32 %1, [%3];\n\t"
        "@p add.u32 %3, %3, 4;\n\t"
        "and.b32 %2, %2, 31;\n\t"
        "}"
        : "+r"(r.hi), "+r"(r.lo), "+r"(r.off), "+r"(r.next)
        : "r"(len)
        : "memory");
}

// Same step for sHAC: the row of the entry comes from the staged slice of ri, x is gathered by row.
template <int kRowBytes, int kRiOffset>
__device__ __forceinline__ void fast_consume_sparse(FastReader& r, uint32_t val, uint32_t len, uint32_t ri_addr,
                                                    uint32_t xs_abs, float& acc) {
    if (kRowBytes == 2) {
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            ".reg .f32 xv;\n\t"
            ".reg .b32 row;\n\t"
            ".reg .b16 r16;\n\t"
            "ld.shared.u16 r16, [%7+%9];\n\t"
            "cvt.u32.u16 row, r16;\n\t"
            "mad.lo.u32 row, row, 4, %8;\n\t"
            "ld.shared.f32 xv, [row];\n\t"
            "add.u32 %2, %2, %6;\n\t"
            "setp.ge.u32 p, %2, 32;\n\t"
            "@p mov.u32 %0, %1;\n\t"
            "@p ld.shared.u32 %1, [%3];\n\t"
            "@p add.u32 %3, %3, 4;\n\t"
            "and.b32 %2, %2, 31;\n\t"
            "fma.rn.f32 %4, xv, %5, %4;\n\t"
            "}"
            : "+r"(r.hi), "+r"(r.lo), "+r"(r.off), "+r"(r.next), "+f"(acc)
            : "f"(__uint_as_float(val)), "r"(len), "r"(ri_addr), "r"(xs_abs), "n"(kRiOffset)
            : "memory");
    } else {
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            ".reg .f32 xv;\n\t"
            ".reg .b32 row;\n\t"
            "ld.shared.u32 row, [%7+%9];\n\t"
            "mad.lo.u32 row, row, 4, %8;\n\t"
            "ld.shared.f32 xv, [row];\n\t"
            "add.u32 %2, %2, %6;\n\t"
            "setp.ge.u32 p, %2, 32;\n\t"
            "@p mov.u32 %0, %1;\n\t"
            "@p ld.shared.u32 %1, [%3];\n\t"
            "@p add.u32 %3, %3, 4;\n\t"
            "and.b32 %2, %2, 31;\n\t"
            "fma.rn.f32 %4, xv, %5, %4;\n\t"
            "}"
            : "+r"(r.hi), "+r"(r.lo), "+r"(r.off), "+r"(r.next), "+f"(acc)
            : "f"(__uint_as_float(val)), "r"(len), "r"(ri_addr), "r"(xs_abs), "n"(kRiOffset)
            : "memory");
    }
}

// ------------------------------------------------------------------------------------------------
// Bulk asynchronous copy global -> shared (TMA, untiled form) with completion on an mbarrier.
// Source, destination and size must be multiples of 16 bytes.  The wait is bounded: it returns
// false if the copy has not landed after kBulkWaitTries polls, and the caller then copies with
// ordinary loads instead.
// ------------------------------------------------------------------------------------------------
constexpr uint32_t kBulkWaitTries = 200000;

__device__ __forceinline__ void mbar_init(uint32_t mbar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(arrivals) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t mbar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t mbar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(mbar)
                 : "memory");
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t mbar, uint32_t parity) {
    for (uint32_t t = 0; t < kBulkWaitTries; ++t) {
        uint32_t done;
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t"
            "}"
            : "=r"(done)
            : "r"(mbar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    return false;
}

// Level-1 entry that stands for a prefix of longer code words: sub-table, then the search.
__device__ __forceinline__ void resolve_long(uint32_t top, const Decoder& d, const DevFormat& f, uint32_t& val,
                                             uint32_t& len) {
    const uint32_t q = (top << d.l1_bits) >> (32 - (len & 31u));
    uint2 e = lds64(d.sub + val + (q << 3));
    if (e.y == 0) e = decode_long(top, f.lut, f.lut_bits, f.rank_value, f.limit, f.first_left, f.rank_base, f.max_len);
    val = e.x; len = e.y;
}

// The same for tables in the split form (see split_entry): lo and hi | length come back.
__device__ __forceinline__ void resolve_long_split(uint32_t top, const Decoder& d, const DevFormat& f, uint32_t& lo,
                                                   uint32_t& hi_len) {
    const uint32_t q = (top << d.l1_bits) >> (32 - (hi_len & 31u));
    uint2 e = lds64(d.sub + lo + (q << 3));
    if (e.y == 0)
        e = split_entry(decode_long(top, f.lut, f.lut_bits, f.rank_value, f.limit, f.first_left, f.rank_base, f.max_len));
    lo = e.x; hi_len = e.y;
}

// First-level entry that does not hold the symbol, for either kind of table.
template <int kTab>
__device__ __forceinline__ void resolve_any(uint32_t top, const Decoder& d, const DevFormat& f, uint32_t& val, uint32_t& len) {
    if (kTab == 0) { resolve_long(top, d, f, val, len); return; }
    const uint2 e = decode_long(top, f.lut, f.lut_bits, f.rank_value, f.limit, f.first_left, f.rank_base, f.max_len);
    val = e.x; len = e.y;
}

// One code word -> the shared value, plain C++ (ragged ends and test paths), for either kind of table.
template <int kTab, bool kLong>
__device__ __forceinline__ float decode_value_any(BitReader& br, const Decoder& d, const DevFormat& f) {
    if (kTab == 0) return decode_value<kLong>(br, d, f);
    const uint32_t top = br.peek();
    const uint32_t idx = (__float_as_uint(__uint2float_rz(~top | d.xt_low)) >> d.l1_shift) - d.bias;
    uint2 e = lds64(d.l1_lane + idx * d.l1_mul);
    if (kLong && (int32_t)e.y < 0)
        e = decode_long(top, f.lut, f.lut_bits, f.rank_value, f.limit, f.first_left, f.rank_base, f.max_len);
    br.skip(e.y);
    return __uint_as_float(e.x);
}

// resolve_long_split for either kind of table.
template <int kTab>
__device__ __forceinline__ void resolve_split_any(uint32_t top, const Decoder& d, const DevFormat& f, uint32_t& lo,
                                                  uint32_t& hi_len) {
    if (kTab == 0) { resolve_long_split(top, d, f, lo, hi_len); return; }
    const uint2 e = split_entry(decode_long(top, f.lut, f.lut_bits, f.rank_value, f.limit, f.first_left, f.rank_base, f.max_len));
    lo = e.x; hi_len = e.y;
}

// N (2 or 3) code words from one window, for tables in the split form {lo, hi | length} (see split_entry):
// as lookup3, with the length taken from the low bits of the second word (the funnel shift only looks at
// its low five bits).  tot = sum of the lengths, flags = kSplitLong if an entry does not hold its symbol.
template <int kTab, int N>
__device__ __forceinline__ void lookup_group_split(const FastReader& r, uint32_t l1_shift, uint32_t l1_mul, uint32_t l1_lane,
                                                   uint32_t xt_low, uint32_t (&wl)[N], uint32_t (&wh)[N], uint32_t& tot,
                                                   uint32_t& flags) {
    uint32_t t;
    const uint32_t zero = 0;
    asm volatile("shf.l.wrap.b32 %0, %1, %2, %3;" : "=r"(t) : "r"(r.lo), "r"(r.hi), "r"(r.off));
#pragma unroll
    for (int i = 0; i < N; ++i) {
        if (kTab == 0) {
            asm volatile(
                "{\n\t.reg .b32 i;\n\t"
                "shr.u32 i, %2, %3;\n\t"
                "mad.lo.u32 i, i, %4, %5;\n\t"
                "ld.shared.v2.u32 {%0, %1}, [i];\n\t}"
                : "=r"(wl[i]), "=r"(wh[i]) : "r"(t), "r"(l1_shift), "r"(l1_mul), "r"(l1_lane) : "memory");
        } else {
            asm volatile(
                "{\n\t.reg .b32 i;\n\t"
                "lop3.b32 i, %2, %6, 0, 0xCF;\n\t"
                "cvt.rz.f32.u32 i, i;\n\t"
                "shr.u32 i, i, %3;\n\t"
                "mad.lo.u32 i, i, %4, %5;\n\t"
                "ld.shared.v2.u32 {%0, %1}, [i];\n\t}"
                : "=r"(wl[i]), "=r"(wh[i]) : "r"(t), "r"(l1_shift), "r"(l1_mul), "r"(l1_lane), "r"(xt_low) : "memory");
        }
        if (i + 1 < N) asm volatile("shf.l.wrap.b32 %0, %1, %0, %2;" : "+r"(t) : "r"(zero), "r"(wh[i]));
    }
    uint32_t sum = wh[0], any = wh[0];
#pragma unroll
    for (int i = 1; i < N; ++i) { sum += wh[i]; any |= wh[i]; }
    tot = sum & 0xffu;
    flags = any & kSplitLong;
}

// One step of kChains chains: lookups first, then the consumes, so that the table loads overlap.
template <bool kLong, int kChains, int kXOffset>
__device__ __forceinline__ void fast_step(FastReader (&r)[kChains], const Decoder& d, const DevFormat& f,
                                          uint32_t l1_lane_abs, const uint32_t (&xa)[kChains], float (&acc)[kChains]) {
    uint32_t top[kChains], val[kChains], len[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) fast_lookup(r[c], d.l1_shift, d.l1_mul, l1_lane_abs, top[c], val[c], len[c]);
    if (kLong) {
#pragma unroll
        for (int c = 0; c < kChains; ++c)
            if ((int32_t)len[c] < 0) resolve_long(top[c], d, f, val[c], len[c]);
    }
#pragma unroll
    for (int c = 0; c < kChains; ++c) fast_consume<kXOffset>(r[c], val[c], len[c], xa[c], acc[c]);
}

// Start bit of each lane's sub-segment inside the segment (exclusive scan of the 32 lengths by
// shuffles) and the segment's total bit length.
__device__ __forceinline__ uint32_t lane_start_bits(uint32_t my_bits, uint32_t lane, uint32_t& total) {
    uint32_t inc = my_bits;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t v = __shfl_up_sync(0xffffffffu, inc, d);
        if ((int)lane >= d) inc += v;
    }
    total = __shfl_sync(0xffffffffu, inc, 31);
    return inc - my_bits;
}

// Programmatic dependent launch.  The product kernels are launched so that they may start while the
// kernel before them in the stream is still draining: everything they read before depends_wait() is
// part of the uploaded format (stream, index, tables), which no kernel writes, so fetching it early is
// safe; x, the workspace and y are touched only after depends_wait(), which returns once the earlier
// kernel has completed and its writes are visible.  allow_dependents() lets the kernel after this one
// do the same.
__device__ __forceinline__ void allow_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void depends_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Asynchronous 16-byte copy global -> shared (both 16-byte aligned); copies_landed() waits for all
// of this thread's copies.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void copies_landed() {
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// Copy the stream span of one segment to the warp's staging area, 16 bytes per lane and request,
// coalesced and asynchronous: the caller waits with copies_landed() and a warp (or block) barrier
// before the lanes read the span.  Returns the bit position of the segment start relative to the
// staged span.
__device__ __forceinline__ uint32_t stage_span(const DevFormat& f, uint64_t seg_bit, uint32_t total_bits,
                                               uint4* stage, uint32_t lane) {
    const uint64_t first_chunk = seg_bit >> 7;
    const uint64_t last_word = ((seg_bit + total_bits) >> 5) + 2;
    const uint32_t chunks = (uint32_t)((last_word >> 2) - first_chunk + 1);
    const uint4* src = reinterpret_cast<const uint4*>(f.stream) + first_chunk;
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(stage);
    for (uint32_t c = lane; c < chunks; c += 32) cp_async16(dst + 16 * c, src + c);
    return (uint32_t)(seg_bit - (first_chunk << 7));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

// ------------------------------------------------------------------------------------------------
// Three code words from one 32-bit window.  The window holds 32 valid bits from the current position,
// so after a code word of length l the next one starts at window << l, and a third one after that,
// as long as the three lengths add up to at most 32; the caller checks `tot` (and `flags`, the OR of
// the three length words, whose top bit marks an entry that does not hold its symbol) before it uses
// the values, and otherwise decodes the three code words one at a time.  The reader is not advanced.
// The asm block hands back the three length words; their sum and OR are formed outside it, so that the
// compiler picks the instructions (one three-input add) and drops `flags` where it is not used.
// ------------------------------------------------------------------------------------------------
template <int kTab>
__device__ __forceinline__ void lookup3(const FastReader& r, uint32_t l1_shift, uint32_t l1_mul, uint32_t l1_lane,
                                        uint32_t xt_low, uint32_t& v1, uint32_t& v2, uint32_t& v3, uint32_t& tot,
                                        uint32_t& flags) {
    uint32_t la, lb, lc;
    if (kTab == 0) {
        asm volatile(
            "{\n\t"
            ".reg .b32 t, i;\n\t"
            "shf.l.wrap.b32 t, %6, %7, %8;\n\t"
            "shr.u32 i, t, %9;\n\t"
            "mad.lo.u32 i, i, %10, %11;\n\t"
            "ld.shared.v2.u32 {%0, %3}, [i];\n\t"
            "shl.b32 t, t, %3;\n\t"
            "shr.u32 i, t, %9;\n\t"
            "mad.lo.u32 i, i, %10, %11;\n\t"
            "ld.shared.v2.u32 {%1, %4}, [i];\n\t"
            "shl.b32 t, t, %4;\n\t"
            "shr.u32 i, t, %9;\n\t"
            "mad.lo.u32 i, i, %10, %11;\n\t"
            "ld.shared.v2.u32 {%2, %5}, [i];\n\t"
            "}"
            : "=r"(v1), "=r"(v2), "=r"(v3), "=r"(la), "=r"(lb), "=r"(lc)
            : "r"(r.lo), "r"(r.hi), "r"(r.off), "r"(l1_shift), "r"(l1_mul), "r"(l1_lane)
            : "memory");
    } else {
        asm volatile(
            "{\n\t"
            ".reg .b32 t, i;\n\t"
            "shf.l.wrap.b32 t, %6, %7, %8;\n\t"
            "lop3.b32 i, t, %12, 0, 0xCF;\n\t"
            "cvt.rz.f32.u32 i, i;\n\t"
            "shr.u32 i, i, %9;\n\t"
            "mad.lo.u32 i, i, %10, %11;\n\t"
            "ld.shared.v2.u32 {%0, %3}, [i];\n\t"
            "shl.b32 t, t, %3;\n\t"
            "lop3.b32 i, t, %12, 0, 0xCF;\n\t"
            "cvt.rz.f32.u32 i, i;\n\t"
            "shr.u32 i, i, %9;\n\t"
            "mad.lo.u32 i, i, %10, %11;\n\t"
            "ld.shared.v2.u32 {%1, %4}, [i];\n\t"
            "shl.b32 t, t, %4;\n\t"
            "lop3.b32 i, t, %12, 0, 0xCF;\n\t"
            "cvt.rz.f32.u32 i, i;\n\t"
            "shr.u32 i, i, %9;\n\t"
            "mad.lo.u32 i, i, %10, %11;\n\t"
            "ld.shared.v2.u32 {%2, %5}, [i];\n\t"
            "}"
            : "=r"(v1), "=r"(v2), "=r"(v3), "=r"(la), "=r"(lb), "=r"(lc)
            : "r"(r.lo), "r"(r.hi), "r"(r.off), "r"(l1_shift), "r"(l1_mul), "r"(l1_lane), "r"(xt_low)
            : "memory");
    }
    tot = la + lb + lc;
    flags = la | lb | lc;
}

// The three code words of lookup3 one at a time (refills in between, entries without a symbol resolved):
// where a lane's three lengths exceed the window, or one of its entries does not hold its symbol.  Rare,
// so it is a call, which keeps the unrolled code around it small.  `sf` is the block's copy of the format
// descriptor in shared memory.
struct Slow3 { uint32_t hi, lo, off, next, v0, v1, v2; };
template <int kTab, bool kLong>
__device__ __noinline__ Slow3 decode3_slow(uint32_t hi, uint32_t lo, uint32_t off, uint32_t next_rel, Decoder dec,
                                           const DevFormat* sf) {
    BitReader br;
    br.hi = hi; br.lo = lo; br.off = off; br.next = next_rel;
    Slow3 r;
    r.v0 = __float_as_uint(decode_value_any<kTab, kLong>(br, dec, *sf));
    r.v1 = __float_as_uint(decode_value_any<kTab, kLong>(br, dec, *sf));
    r.v2 = __float_as_uint(decode_value_any<kTab, kLong>(br, dec, *sf));
    r.hi = br.hi; r.lo = br.lo; r.off = br.off; r.next = br.next;
    return r;
}

// Advance the reader by up to 32 bits (one refill at most).
__device__ __forceinline__ void fast_advance(FastReader& r, uint32_t bits) { fast_consume_value(r, bits); }

// ------------------------------------------------------------------------------------------------
// HAC, one input vector (Algorithm 1 by segments).  x is staged in shared memory; a lane's rows
// are consecutive, lanes are S rows apart, so one padding word per sub-segment (when S is even)
// keeps the 32 lanes on distinct banks.
//   kMode 0: product; 1: debug decode (values written to out[j*n + i]).
// ------------------------------------------------------------------------------------------------
//   kGroup: code words are decoded three to a window (lookup3), from either kind of first-level table (kTab);
//           kGuard: three lengths can exceed the window.  Without kGroup the table is the prefix table.
template <int kMode, bool kXShared, bool kLong, int kChains, bool kRuns, bool kGroup = false, int kTab = 0, bool kGuard = false>
__global__ void __launch_bounds__(1024) hac_vec_kernel(DevFormat f, TablePlan tp, const float* __restrict__ x,
                                                       int64_t xs_i, float* __restrict__ y, int64_t ys_j,
                                                       float* __restrict__ aux) {
    // A warp works on kChains consecutive segments at a time (an "item"); every lane then runs
    // kChains independent decode chains, which hides the latency of the dependent table lookups.
    __shared__ DevFormat sf;               // for the rare paths that are calls (decode3_slow)
    if (kGroup && threadIdx.x == 0) sf = f;
    allow_dependents();
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
    const uint32_t items = (f.units + kChains - 1) / kChains;
    // index entries of this warp's first item: requested before the tables are staged so that the
    // trips to memory overlap
    uint32_t item = blockIdx.x + gridDim.x * warp;
    uint32_t my_bits[kChains];
    uint64_t seg_bit[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) {
        const uint32_t u = item * kChains + c;
        my_bits[c] = 0; seg_bit[c] = 0;
        if (item < items && u < f.units) {
            my_bits[c] = __ldg(f.sub_bits + (size_t)u * 32 + lane);
            seg_bit[c] = __ldg(f.seg_bit_off + u);
        }
    }
    // The layout of shared memory is known up front: [tables][x][staging areas].  The first item's spans
    // are requested (asynchronous copies) before the tables and x are staged, so that the block pays one
    // trip to memory for all three.
    const uint32_t pad = (f.S & 1u) ? 0u : 1u;
    const size_t table_bytes = plan_smem_bytes(f.l1_entries, tp.repl_log2, f.sub_bytes);
    const size_t x_bytes = (kMode == 0 && kXShared) ? align16(((size_t)f.n + (f.n / f.S + 1) * pad) * 4) : 0;
    uint4* stage = reinterpret_cast<uint4*>(smem + table_bytes + x_bytes) + (size_t)warp * kChains * f.max_unit_chunks;
    const uint32_t stage_a = smem_off(stage);
    uint32_t start[kChains], base[kChains];
    auto fetch = [&]() {
#pragma unroll
        for (int c = 0; c < kChains; ++c) {
            uint32_t total;
            start[c] = lane_start_bits(my_bits[c], lane, total);
            base[c] = 0;
            if (item * kChains + c < f.units)
                base[c] = stage_span(f, seg_bit[c], total, stage + (size_t)c * f.max_unit_chunks, lane);
        }
    };
    if (item < items) fetch();
    // everything above (index, spans of the first item, tables) reads the format only; x and the outputs
    // belong to the kernels before this one
    depends_wait();
    // the first elements of x are requested together with the tables (one trip to memory for both)
    constexpr int kXAhead = 4;
    float x_v[kXAhead];
    if (kMode == 0 && kXShared) {
#pragma unroll
        for (int k = 0; k < kXAhead; ++k) {
            const uint32_t i = threadIdx.x + k * blockDim.x;
            x_v[k] = i < f.n ? __ldg(x + (int64_t)i * xs_i) : 0.0f;
        }
    }
    unsigned char* p = smem;
    const Decoder dec = stage_decoder(f, tp, p);
    float* xs = reinterpret_cast<float*>(p);
    if (kMode == 0 && kXShared) {
#pragma unroll
        for (int k = 0; k < kXAhead; ++k) {
            const uint32_t i = threadIdx.x + k * blockDim.x;
            if (i < f.n) xs[i + pad * (i / f.S)] = x_v[k];
        }
#pragma unroll 4
        for (uint32_t i = threadIdx.x + kXAhead * blockDim.x; i < f.n; i += blockDim.x)
            xs[i + pad * (i / f.S)] = __ldg(x + (int64_t)i * xs_i);
    }
    const uint32_t xs_a = smem_off(xs);
    __syncthreads();                       // tables and x are in place
    copies_landed();                       // a warp starts as soon as its own spans have landed
    __syncwarp();

    while (item < items) {
        BitReader br[kChains];
        uint32_t count[kChains], xa[kChains];
        float* out[kChains];
        uint32_t common = f.S;
#pragma unroll
        for (int c = 0; c < kChains; ++c) {
            const uint32_t u = item * kChains + c;
            const uint32_t j = u / f.G, g = u - j * f.G;
            const uint32_t sub = g * 32 + lane;              // sub-segment number inside the column
            const uint32_t row0 = sub * f.S;
            count[c] = (u < f.units && row0 < f.n) ? min(f.S, f.n - row0) : 0u;
            common = min(common, count[c]);
            xa[c] = xs_a + ((row0 + pad * sub) << 2);
            out[c] = aux + (size_t)j * f.n + row0;
            br[c].init(stage_a + c * f.max_unit_chunks * 16, base[c] + start[c]);
        }
        // index entries of the next item, in flight while this one is decoded
        const uint32_t next_item = item + gridDim.x * warps;
#pragma unroll
        for (int c = 0; c < kChains; ++c) {
            const uint32_t u = next_item * kChains + c;
            if (next_item < items && u < f.units) {
                my_bits[c] = __ldg(f.sub_bits + (size_t)u * 32 + lane);
                seg_bit[c] = __ldg(f.seg_bit_off + u);
            } else {
                my_bits[c] = 0;
            }
        }
        float acc[kChains];
#pragma unroll
        for (int c = 0; c < kChains; ++c) acc[c] = 0.0f;
        if (kMode == 0 && kXShared && kRuns) {
            // zero-run table: one lookup covers a run of zero entries and the non-zero entry after it
            const uint32_t sb = shared_base();
            const uint32_t l1_abs = sb + dec.l1_lane;
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                FastReader fr;
                fr.hi = br[c].hi; fr.lo = br[c].lo; fr.off = br[c].off; fr.next = sb + br[c].next;
                uint32_t left = count[c], xat = xa[c];
                while (left > 0) {
                    uint32_t top, val, meta;
                    fast_lookup(fr, dec.l1_shift, dec.l1_mul, l1_abs, top, val, meta);
                    uint32_t covered = 1;
                    if ((int32_t)meta < 0) {
                        resolve_long(top, dec, f, val, meta);
                    } else {
                        covered = meta >> 8;
                        meta &= 0xffu;
                        if (covered > left) { covered = 1; meta = tp.zero_len; val = 0u; }   // the run crosses the end: take one zero
                    }
                    fast_consume_value(fr, meta);
                    xat += covered << 2;
                    acc[c] = fmaf(ldsf(xat - 4), __uint_as_float(val), acc[c]);
                    left -= covered;
                }
            }
        } else if (kMode == 0 && kXShared && kGroup) {
            const uint32_t sb = shared_base();
            FastReader fr[kChains];
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                fr[c].hi = br[c].hi; fr[c].lo = br[c].lo; fr[c].off = br[c].off; fr[c].next = sb + br[c].next;
            }
            const uint32_t l1_abs = sb + dec.l1_lane - dec.bias * dec.l1_mul;
            uint32_t s = 0;
            for (; s + 3 <= common; s += 3) {
                uint32_t v[kChains][3], tot[kChains], flags[kChains];
#pragma unroll
                for (int c = 0; c < kChains; ++c)
                    lookup3<kTab>(fr[c], dec.l1_shift, dec.l1_mul, l1_abs, dec.xt_low, v[c][0], v[c][1], v[c][2], tot[c], flags[c]);
                if (kGuard || kLong) {
                    bool bad = false;
#pragma unroll
                    for (int c = 0; c < kChains; ++c) bad = bad || (kGuard && tot[c] > 32u) || (kLong && (int32_t)flags[c] < 0);
                    if (__any_sync(__activemask(), bad)) {
                        if (bad) {
#pragma unroll
                            for (int c = 0; c < kChains; ++c) {
                                const Slow3 r = decode3_slow<kTab, kLong>(fr[c].hi, fr[c].lo, fr[c].off, fr[c].next - sb, dec, &sf);
                                fr[c].hi = r.hi; fr[c].lo = r.lo; fr[c].off = r.off; fr[c].next = sb + r.next;
                                v[c][0] = r.v0; v[c][1] = r.v1; v[c][2] = r.v2;
                                tot[c] = 0;
                            }
                        }
                    }
                }
#pragma unroll
                for (int c = 0; c < kChains; ++c) {
                    fast_advance(fr[c], tot[c]);
#pragma unroll
                    for (int e = 0; e < 3; ++e) acc[c] = fmaf(ldsf(xa[c] + 4 * e), __uint_as_float(v[c][e]), acc[c]);
                    xa[c] += 12;
                }
            }
#pragma unroll
            for (int c = 0; c < kChains; ++c) {              // what is left of each chain, one code word at a time
                br[c].hi = fr[c].hi; br[c].lo = fr[c].lo; br[c].off = fr[c].off; br[c].next = fr[c].next - sb;
                for (uint32_t t = s; t < count[c]; ++t) {
                    const float w = decode_value_any<kTab, kLong>(br[c], dec, f);
                    acc[c] = fmaf(ldsf(xa[c]), w, acc[c]);
                    xa[c] += 4;
                }
            }
        } else if (kMode == 0 && kXShared) {
            const uint32_t sb = shared_base();
            FastReader fr[kChains];
            uint32_t xabs[kChains];
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                fr[c].hi = br[c].hi; fr[c].lo = br[c].lo; fr[c].off = br[c].off; fr[c].next = sb + br[c].next;
                xabs[c] = sb + xa[c];
            }
            const uint32_t l1_abs = sb + dec.l1_lane;
            uint32_t s = 0;
            for (; s + 4 <= common; s += 4) {
                fast_step<kLong, kChains, 0>(fr, dec, f, l1_abs, xabs, acc);
                fast_step<kLong, kChains, 4>(fr, dec, f, l1_abs, xabs, acc);
                fast_step<kLong, kChains, 8>(fr, dec, f, l1_abs, xabs, acc);
                fast_step<kLong, kChains, 12>(fr, dec, f, l1_abs, xabs, acc);
#pragma unroll
                for (int c = 0; c < kChains; ++c) xabs[c] += 16;
            }
            for (; s < common; ++s) {
                fast_step<kLong, kChains, 0>(fr, dec, f, l1_abs, xabs, acc);
#pragma unroll
                for (int c = 0; c < kChains; ++c) xabs[c] += 4;
            }
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                br[c].hi = fr[c].hi; br[c].lo = fr[c].lo; br[c].off = fr[c].off; br[c].next = fr[c].next - sb;
                xa[c] = xabs[c] - sb;
                for (uint32_t t = common; t < count[c]; ++t) {
                    const float w = decode_value<kLong>(br[c], dec, f);
                    acc[c] = fmaf(ldsf(xa[c]), w, acc[c]);
                    xa[c] += 4;
                }
            }
        } else if (kMode == 0) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                const uint32_t u = item * kChains + c;
                const uint32_t j = u / f.G, g = u - j * f.G;
                const float* xl = x + (int64_t)((g * 32 + lane) * f.S) * xs_i;
                for (uint32_t s = 0; s < count[c]; ++s) {
                    const float w = decode_value<kLong>(br[c], dec, f);
                    acc[c] = fmaf(xl[(int64_t)s * xs_i], w, acc[c]);
                }
            }
        } else {
#pragma unroll
            for (int c = 0; c < kChains; ++c)
                for (uint32_t s = 0; s < count[c]; ++s) out[c][s] = decode_value<kLong>(br[c], dec, f);
        }
        if (kMode == 0) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) acc[c] = warp_sum(acc[c]);
            if (lane == 0) {
                if (kChains == 2 && f.G == 2) {              // the item is one whole column
                    y[(int64_t)item * ys_j] = finish_output(f, acc[0] + acc[kChains - 1], item);
                } else {
#pragma unroll
                    for (int c = 0; c < kChains; ++c) {
                        const uint32_t u = item * kChains + c;
                        if (u < f.units) {
                            if (f.G == 1) y[(int64_t)u * ys_j] = finish_output(f, acc[c], u);
                            else aux[u] = acc[c];
                        }
                    }
                }
            }
        }
        __syncwarp();
        item = next_item;
        if (item < items) {
            fetch();
            copies_landed();
            __syncwarp();
        }
    }
}

// ------------------------------------------------------------------------------------------------
// HAC, one input vector, rows held in registers (Algorithm 1 by segments).
//
// A column of W is G segments of 32 sub-segments of kS rows.  Here a warp does not walk down a column:
// it keeps ONE segment position g ("class") for its whole life, i.e. lane l always multiplies rows
// (32 g + l) kS .. + kS - 1, so it loads those kS elements of x into registers once and then decodes
// that segment of one column after another.  The multiply-accumulate of a decoded symbol is then a
// single FMA with a register operand: no shared-memory read of x per symbol.  A block owns a
// contiguous range of columns; its warps are dealt round-robin to the classes, and the warps of a
// class take the block's columns kC at a time (kC interleaved decode chains per lane, all on the
// same rows).  Per-segment sums meet in shared memory and are added per column in segment order at
// the end, so no second kernel and no workspace is needed whatever G is.
//
// Code words are decoded three to a window (lookup3): one window extraction and one refill test per
// three symbols.  A lane whose three lengths exceed the window, or that meets an entry without its
// symbol, leaves the unrolled code and finishes its sub-segment one code word at a time.
//
// Order in a block: index entries of the first two items and the table entries are requested together
// (optionally also the block's range of the stream into L2); the spans of the first item are requested
// and the tables staged BEFORE the dependency wait, since all of that is format data; x follows the
// wait; the spans of a warp's next item are copied to shared memory (cp.async, second buffer set) while
// the current item is decoded.
//   kMode 0: product; 1: debug decode (values written to aux[j*n + i]).
//   kTab  0: prefix table; 1: magnitude table.   kGuard: three lengths can exceed 32 bits.
// ------------------------------------------------------------------------------------------------
template <int kMode, int kS, int kC, int kTab, bool kLong, bool kGuard>
__global__ void __launch_bounds__(kC <= 2 ? 512 : 384, 1) hac_rows_kernel(DevFormat f, TablePlan tp, const float* __restrict__ x,
                                                          int64_t xs_i, float* __restrict__ y, int64_t ys_j,
                                                          float* __restrict__ aux, uint32_t colsum_bytes,
                                                          uint32_t stream_chunks) {
    __shared__ DevFormat sf;               // for the rare paths that are calls (decode3_slow)
    allow_dependents();
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
    const uint32_t col0 = (uint32_t)(((uint64_t)f.m * blockIdx.x) / gridDim.x);
    const uint32_t col1 = (uint32_t)(((uint64_t)f.m * (blockIdx.x + 1)) / gridDim.x);
    const uint32_t ncol = col1 - col0;
    if (threadIdx.x == 0) sf = f;
    const uint32_t cls = warp % f.G, wrank = warp / f.G;            // the host launches at least G warps
    const uint32_t wcls = (warps - cls + f.G - 1) / f.G;            // warps of this class
    const uint32_t groups = (ncol + kC - 1) / kC;
    const uint32_t nitems = wrank < groups ? (groups - wrank + wcls - 1) / wcls : 0u;
    const uint32_t sub = cls * 32 + lane;                           // sub-segment number inside a column
    const uint32_t row0 = sub * kS;
    const uint32_t count = row0 < f.n ? min((uint32_t)kS, f.n - row0) : 0u;

    // shared memory: [tables][per-column partial sums][span buffers: set, warp, chain]; x is staged over the
    // second buffer set before that set is first used
    const size_t table_bytes = plan_smem_bytes(f.l1_entries, tp.repl_log2, f.sub_bytes);
    float* colsum = reinterpret_cast<float*>(smem + table_bytes);
    const uint32_t span_bytes = f.max_unit_chunks * 16;
    const uint32_t bufs = (uint32_t)table_bytes + colsum_bytes;
    const uint32_t set_bytes = warps * kC * span_bytes;
    float* xs = reinterpret_cast<float*>(smem + bufs + set_bytes);
    auto buf_of = [&](uint32_t set, uint32_t c) { return bufs + set * set_bytes + (warp * kC + c) * span_bytes; };

    // index entries of item k of this warp (chain c = column (wrank + k wcls) kC + c of the block)
    auto col_of = [&](uint32_t k, uint32_t c) { return col0 + (wrank + k * wcls) * kC + c; };
    struct Index { uint32_t bits[kC]; uint64_t seg[kC]; };
    auto load_index = [&](uint32_t k, Index& ix) {
        if (k >= nitems) return;
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            const uint32_t col = col_of(k, c);
            ix.bits[c] = 0; ix.seg[c] = 0;
            if (col < col1) {
                const size_t u = (size_t)col * f.G + cls;
                ix.bits[c] = __ldg(f.sub_bits + u * 32 + lane);
                ix.seg[c] = __ldg(f.seg_bit_off + u);
            }
        }
    };
    // requests the spans of item k into buffer set `set`; pos[c] = bit position (relative to the buffer of
    // chain c) of this lane's first code word.  Always one commit group.
    auto fetch = [&](uint32_t k, uint32_t set, const Index& ix, uint32_t (&pos)[kC]) {
        if (k < nitems) {
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                uint32_t total;
                const uint32_t start = lane_start_bits(ix.bits[c], lane, total);
                pos[c] = 0;
                if (col_of(k, c) < col1)
                    pos[c] = start + stage_span(f, ix.seg[c], total, reinterpret_cast<uint4*>(smem + buf_of(set, c)), lane);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    uint32_t pos_cur[kC], pos_nxt[kC];
    Index ix0, ix1;
    load_index(0, ix0);
    load_index(1, ix1);
    // table entries: every warp takes groups of 32 consecutive entries, all its loads in flight at once
    constexpr int kTabAhead = 4;
    const uint32_t entries = f.l1_entries;
    uint2 te[kTabAhead];
#pragma unroll
    for (int i = 0; i < kTabAhead; ++i) {
        const uint32_t idx = (warp + i * warps) * 32 + lane;
        te[i] = idx < entries ? __ldg(f.l1 + idx) : make_uint2(0u, 0u);
    }
    if (tp.prefetch) {
        // the block's share of the stream, a little generously, towards L2: 16 KB per requesting thread
        const uint32_t lo = (uint32_t)(((uint64_t)stream_chunks * col0) / f.m);
        const uint32_t hi = (uint32_t)(((uint64_t)stream_chunks * col1) / f.m);
        const uint32_t slack = 64 + ((hi - lo) >> 6);
        const uint32_t from = lo > slack ? lo - slack : 0u, to = min(stream_chunks, hi + slack);
        const uint32_t piece = 1024;
        const uint32_t at = from + threadIdx.x * piece;
        if (at < to) {
            const uint32_t bytes = min(piece, to - at) * 16u;
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(reinterpret_cast<const uint4*>(f.stream) + at),
                         "r"(bytes)
                         : "memory");
        }
    }
    fetch(0, 0, ix0, pos_cur);
    // tables -> shared memory, replicated (see TablePlan): the warp writes its 32 entries' replicas slot by
    // slot, the value for a slot fetched from the lane that holds it (consecutive lanes write consecutive slots)
    Decoder dec;
    {
        uint2* l1 = reinterpret_cast<uint2*>(smem);
        uint2* subt = reinterpret_cast<uint2*>(smem + (((size_t)8 * f.l1_entries) << tp.repl_log2));
        const uint32_t repl = 1u << tp.repl_log2;
        auto spread = [&](uint32_t idx0, uint2 v) {
            uint2* dst = l1 + ((size_t)idx0 << tp.repl_log2);
            const uint32_t warp_slots = min(32u, entries - idx0) << tp.repl_log2;
            for (uint32_t s0 = 0; s0 < warp_slots; s0 += 32) {
                const uint32_t src = (s0 + lane) >> tp.repl_log2;
                uint2 w;
                w.x = __shfl_sync(0xffffffffu, v.x, src & 31u);
                w.y = __shfl_sync(0xffffffffu, v.y, src & 31u);
                if (s0 + lane < warp_slots) dst[s0 + lane] = w;
            }
        };
#pragma unroll
        for (int i = 0; i < kTabAhead; ++i) {
            const uint32_t idx0 = (warp + i * warps) * 32;
            if (idx0 < entries) spread(idx0, te[i]);
        }
        for (uint32_t idx0 = (warp + kTabAhead * warps) * 32; idx0 < entries; idx0 += warps * 32) {
            const uint32_t idx = idx0 + lane;
            spread(idx0, idx < entries ? __ldg(f.l1 + idx) : make_uint2(0u, 0u));
        }
        for (uint32_t i = threadIdx.x; i < f.sub_bytes / 8; i += blockDim.x) subt[i] = __ldg(f.sub + i);
        dec.l1_lane = smem_off(l1) + ((threadIdx.x & (repl - 1)) << 3);
        dec.l1_mul = 8u << tp.repl_log2;
        dec.l1_shift = f.tab_kind ? 23 - f.xt_mant : 32 - f.l1_bits;
        dec.bias = f.tab_kind ? (127u + f.xt_row0) << f.xt_mant : 0u;
        dec.xt_low = f.xt_low;
        dec.l1_bits = f.l1_bits;
        dec.sub = smem_off(subt);
    }
    // everything above (index, spans of the first item, tables) reads the format only; x and the outputs
    // belong to the kernels before this one
    depends_wait();
    float xr[kS];
    constexpr int kXAhead = 8;
    const uint32_t rows = f.G * 32u * kS;
    float xv[kXAhead];
    if (kMode == 0) {                      // the first elements of x, all requests in flight at once
#pragma unroll
        for (int i = 0; i < kXAhead; ++i) {
            const uint32_t r = threadIdx.x + i * blockDim.x;
            xv[i] = r < f.n ? __ldg(x + (int64_t)r * xs_i) : 0.0f;
        }
    }
    if (kMode == 0) {
        // x -> shared memory (coalesced; one padding word per sub-segment keeps the lanes of a warp, which
        // are kS rows apart, on distinct banks; rows past the end of x are zeros) -> registers
        for (uint32_t r0 = 0; r0 < rows; r0 += kXAhead * blockDim.x) {
            if (r0 > 0) {
#pragma unroll
                for (int i = 0; i < kXAhead; ++i) {
                    const uint32_t r = r0 + threadIdx.x + i * blockDim.x;
                    xv[i] = r < f.n ? __ldg(x + (int64_t)r * xs_i) : 0.0f;
                }
            }
#pragma unroll
            for (int i = 0; i < kXAhead; ++i) {
                const uint32_t r = r0 + threadIdx.x + i * blockDim.x;
                if (r < rows) xs[r + r / kS] = xv[i];
            }
        }
        __syncthreads();
#pragma unroll
        for (int s = 0; s < kS; ++s) xr[s] = xs[row0 + sub + s];
    }
    __syncthreads();                       // tables are in place; x has left the second buffer set
    fetch(1, 1, ix1, pos_nxt);
    load_index(2, ix0);

    const uint32_t sb = shared_base();
    const uint32_t l1_abs = sb + dec.l1_lane - dec.bias * dec.l1_mul;
    for (uint32_t k = 0; k < nitems; ++k) {
        const uint32_t set = k & 1u;
        asm volatile("cp.async.wait_group 1;" ::: "memory");      // item k's spans (item k + 1's may be in flight)
        __syncwarp();
        bool has[kC];
        uint32_t bufc[kC];
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            has[c] = col_of(k, c) < col1;
            bufc[c] = buf_of(set, has[c] ? c : 0);                  // a chain without a column decodes chain 0's again
            if (!has[c]) pos_cur[c] = pos_cur[0];
        }
        float acc[kC];
#pragma unroll
        for (int c = 0; c < kC; ++c) acc[c] = 0.0f;
        if (count > 0) {
            FastReader fr[kC];
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                BitReader br;
                br.init(bufc[c], pos_cur[c]);
                fr[c].hi = br.hi; fr[c].lo = br.lo; fr[c].off = br.off; fr[c].next = sb + br.next;
            }
            float* out[kC];
            if (kMode == 1) {
#pragma unroll
                for (int c = 0; c < kC; ++c) out[c] = aux + (size_t)col_of(k, c) * f.n + row0;
            }
            uint32_t done = 0;                                      // symbols of the sub-segment finished by the unrolled code
            if (count == kS) {
#pragma unroll
                for (int s = 0; s + 3 <= kS; s += 3) {
                    uint32_t v[kC][3], tot[kC], flags[kC];
#pragma unroll
                    for (int c = 0; c < kC; ++c)
                        lookup3<kTab>(fr[c], dec.l1_shift, dec.l1_mul, l1_abs, dec.xt_low, v[c][0], v[c][1], v[c][2], tot[c], flags[c]);
                    if (kGuard || kLong) {
                        // one test for all chains: the OR of the sums is above 32 if one of them is (and, rarely,
                        // when one is exactly 32: the slow path is right for any group); only the lanes concerned
                        // leave the unrolled code
                        uint32_t tall = 0, fall = 0;
#pragma unroll
                        for (int c = 0; c < kC; ++c) { tall |= tot[c]; fall |= flags[c]; }
                        const bool bad = (kGuard && tall > 32u) || (kLong && (int32_t)fall < 0);
                        {
                            if (bad) {
#pragma unroll
                                for (int c = 0; c < kC; ++c) {
                                    const Slow3 r = decode3_slow<kTab, kLong>(fr[c].hi, fr[c].lo, fr[c].off, fr[c].next - sb, dec, &sf);
                                    fr[c].hi = r.hi; fr[c].lo = r.lo; fr[c].off = r.off; fr[c].next = sb + r.next;
                                    v[c][0] = r.v0; v[c][1] = r.v1; v[c][2] = r.v2;
                                    tot[c] = 0;
                                }
                            }
                        }
                    }
#pragma unroll
                    for (int c = 0; c < kC; ++c) {
                        fast_advance(fr[c], tot[c]);
#pragma unroll
                        for (int e = 0; e < 3; ++e) {
                            if (kMode == 0) acc[c] = fmaf(xr[s + e], __uint_as_float(v[c][e]), acc[c]);
                            else if (has[c]) out[c][s + e] = __uint_as_float(v[c][e]);
                        }
                    }
                }
#pragma unroll
                for (int s = kS - kS % 3; s < kS; ++s) {            // the symbols that do not fill a group of three
                    uint32_t top[kC], val[kC], len[kC];
#pragma unroll
                    for (int c = 0; c < kC; ++c) table_lookup<kTab>(fr[c], dec.l1_shift, dec.l1_mul, l1_abs, dec.xt_low, top[c], val[c], len[c]);
                    if (kLong) {
#pragma unroll
                        for (int c = 0; c < kC; ++c)
                            if ((int32_t)len[c] < 0) resolve_any<kTab>(top[c], dec, f, val[c], len[c]);
                    }
#pragma unroll
                    for (int c = 0; c < kC; ++c) {
                        fast_advance(fr[c], len[c]);
                        if (kMode == 0) acc[c] = fmaf(xr[s], __uint_as_float(val[c]), acc[c]);
                        else if (has[c]) out[c][s] = __uint_as_float(val[c]);
                    }
                }
                done = (uint32_t)kS;
            }
            if (done < count) {
                // the sub-segment at the ragged end of a column
#pragma unroll
                for (int c = 0; c < kC; ++c) {
                    BitReader br;
                    br.hi = fr[c].hi; br.lo = fr[c].lo; br.off = fr[c].off; br.next = fr[c].next - sb;
                    for (uint32_t s = done; s < count; ++s) {
                        const float w = decode_value_any<kTab, kLong>(br, dec, f);
                        if (kMode == 0) acc[c] = fmaf(__ldg(x + (int64_t)(row0 + s) * xs_i), w, acc[c]);
                        else if (has[c]) out[c][s] = w;
                    }
                }
            }
        }
        __syncwarp();
        if (kMode == 0) {
#pragma unroll
            for (int c = 0; c < kC; ++c) acc[c] = warp_sum(acc[c]);
            if (lane == 0) {
#pragma unroll
                for (int c = 0; c < kC; ++c)
                    if (has[c]) colsum[(col_of(k, c) - col0) * f.G + cls] = acc[c];
            }
        }
        // the buffer set just decoded takes the spans of item k + 2
#pragma unroll
        for (int c = 0; c < kC; ++c) pos_cur[c] = pos_nxt[c];
        fetch(k + 2, set, ix0, pos_nxt);
        load_index(k + 3, ix0);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (kMode == 0) {
        __syncthreads();
        for (uint32_t t = threadIdx.x; t < ncol; t += blockDim.x) {
            float s = 0.0f;
            for (uint32_t g = 0; g < f.G; ++g) s += colsum[t * f.G + g];
            y[(int64_t)(col0 + t) * ys_j] = finish_output(f, s, col0 + t);
        }
    }
}

// Work item of the sHAC single-input kernel (derived on the host from cb and the offset index): one
// or two consecutive segments of one column.  For each segment: where its code words start in the
// stream, where its entries start in nz / ri, and how many there are.
struct ShacItem {
    uint64_t bit_off[2];
    uint32_t pos0[2], count[2];
    uint32_t col, segments, whole_column, first_unit;
};

__device__ __forceinline__ ShacItem load_item(const void* base, uint32_t index) {     // header of a kItemWords record
    const uint4* w = reinterpret_cast<const uint4*>(base) + (size_t)index * (kItemWords / 4);
    const uint4 a = __ldg(w), b = __ldg(w + 1), c = __ldg(w + 2);
    ShacItem r;
    r.bit_off[0] = ((uint64_t)a.y << 32) | a.x; r.pos0[0] = a.z; r.count[0] = a.w;
    r.bit_off[1] = ((uint64_t)b.y << 32) | b.x; r.pos0[1] = b.z; r.count[1] = b.w;
    r.col = c.x; r.segments = c.y & 0xffu; r.whole_column = (c.y >> 8) & 1u; r.first_unit = c.z;
    return r;
}

// ------------------------------------------------------------------------------------------------
// sHAC, one input vector (Algorithm 2 by segments): as the HAC kernel over the stored entries of a
// column, with the row of each entry taken from ri (the segment's slice of ri is staged in shared
// memory by coalesced loads) and x gathered from shared memory.  A warp takes one item (up to two
// segments of a column) at a time, so every lane runs two independent decode chains.
// ------------------------------------------------------------------------------------------------
template <int kMode, bool kXShared, bool kLong, typename RowT>
__global__ void __launch_bounds__(1024) shac_vec_kernel(DevFormat f, TablePlan tp, const float* __restrict__ x,
                                                        int64_t xs_i, float* __restrict__ y, int64_t ys_j,
                                                        float* __restrict__ aux) {
    constexpr int kChains = 2;
    constexpr int kRow = (int)sizeof(RowT);
    allow_dependents();
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
    uint32_t item = blockIdx.x + gridDim.x * warp;
    uint32_t my_bits[kChains] = {0, 0};
    ShacItem info;
    info.segments = 0;
    auto load_index = [&](uint32_t it) {
        info = load_item(f.unit_info, it);
#pragma unroll
        for (int c = 0; c < kChains; ++c)
            my_bits[c] = (uint32_t)c < info.segments ? __ldg(f.sub_bits + (size_t)(info.first_unit + c) * 32 + lane) : 0u;
    };
    if (item < f.items) load_index(item);
    unsigned char* p = smem;
    // x: one bulk asynchronous copy when it is contiguous and aligned (it overlaps the table fill
    // and the first segment fetch), ordinary loads otherwise
    const uint32_t mbar = shared_base();
    p += 16;
    float* xs = reinterpret_cast<float*>(p);
    const bool bulk = kMode == 0 && kXShared && tp.x_bulk;
    const uint32_t bulk_bytes = (f.n & ~3u) * 4u;
    if (kMode == 0 && kXShared) p += align16((size_t)f.n * 4);
    if (bulk && threadIdx.x == 0) mbar_init(mbar, 1);
    // [tables] follow at p; the staging areas come after them.  The first item's slices of ri and spans of
    // the stream are requested (asynchronous copies) before the tables are staged, so that the trips to
    // memory overlap.
    unsigned char* after_tables = p + plan_smem_bytes(f.l1_entries, tp.repl_log2, f.sub_bytes);
    uint4* stage = reinterpret_cast<uint4*>(after_tables) + (size_t)warp * kChains * f.max_unit_chunks;
    after_tables += align16((size_t)warps * kChains * f.max_unit_chunks * 16);
    // row-index staging: 32*S entries plus up to 16 bytes of misalignment, per segment
    const uint32_t ri_chunks = (32u * f.S * (uint32_t)kRow + 15u) / 16u + 1u;
    uint4* ri_stage = reinterpret_cast<uint4*>(after_tables) + (size_t)warp * kChains * ri_chunks;
    const uint32_t stage_a = smem_off(stage), ri_a = smem_off(ri_stage), xs_a = smem_off(xs);
    const RowT* __restrict__ ri = reinterpret_cast<const RowT*>(f.ri);

    // requests each segment's slice of ri and its span of the stream (copies_landed() and a barrier
    // come before they are read)
    uint32_t start[kChains], base[kChains], ri_lane[kChains];
    auto fetch = [&]() {
#pragma unroll
        for (int c = 0; c < kChains; ++c) {
            uint32_t total;
            start[c] = lane_start_bits(my_bits[c], lane, total);
            base[c] = 0; ri_lane[c] = ri_a;
            if ((uint32_t)c < info.segments) {
                if (kMode == 0) {
                    const uintptr_t byte0 = reinterpret_cast<uintptr_t>(ri + info.pos0[c]);
                    const uintptr_t chunk0 = byte0 & ~(uintptr_t)15;
                    const uint32_t chunks = (uint32_t)((byte0 + (uintptr_t)info.count[c] * kRow - chunk0 + 15) >> 4);
                    const uint4* src = reinterpret_cast<const uint4*>(chunk0);
                    const uint32_t dst = shared_base() + ri_a + c * ri_chunks * 16;
                    for (uint32_t k = lane; k < chunks; k += 32) cp_async16(dst + 16 * k, src + k);
                    ri_lane[c] = ri_a + c * ri_chunks * 16 + (uint32_t)(byte0 - chunk0) + lane * f.S * (uint32_t)kRow;
                }
                base[c] = stage_span(f, info.bit_off[c], total, stage + (size_t)c * f.max_unit_chunks, lane);
            }
        }
    };
    if (item < f.items) fetch();
    // everything above (index, spans of the first item, tables) reads the format only; x and the outputs
    // belong to the kernels before this one
    depends_wait();
    if (bulk) {
        __syncthreads();                   // the mbarrier is initialised
        if (threadIdx.x == 0 && bulk_bytes > 0) {
            mbar_expect_tx(mbar, bulk_bytes);
            bulk_copy_g2s(shared_base() + smem_off(xs), x, bulk_bytes, mbar);
        }
        for (uint32_t i = (f.n & ~3u) + threadIdx.x; i < f.n; i += blockDim.x) xs[i] = x[i];
    }
    const Decoder dec = stage_decoder(f, tp, p);
    if (kMode == 0 && kXShared && !bulk) {
#pragma unroll 8
        for (uint32_t i = threadIdx.x; i < f.n; i += blockDim.x) xs[i] = __ldg(x + (int64_t)i * xs_i);
    }
    if (bulk) {
        const bool landed = bulk_bytes == 0 || mbar_wait_bounded(mbar, 0);
        if (__syncthreads_or(landed ? 0 : 1)) {             // late or lost: copy x the ordinary way
            for (uint32_t i = threadIdx.x; i < f.n; i += blockDim.x) xs[i] = x[i];
        }
    }
    __syncthreads();                       // tables and x are in place
    copies_landed();                       // a warp starts as soon as its own slices and spans have landed
    __syncwarp();

    while (item < f.items) {
        const ShacItem cur = info;
        BitReader br[kChains];
        uint32_t count[kChains];
        uint32_t common = f.S;
        const uint32_t lane_pos = lane * f.S;
#pragma unroll
        for (int c = 0; c < kChains; ++c) {
            count[c] = ((uint32_t)c < cur.segments && lane_pos < cur.count[c]) ? min(f.S, cur.count[c] - lane_pos) : 0u;
            common = min(common, count[c]);
            br[c].init(stage_a + c * f.max_unit_chunks * 16, base[c] + start[c]);
        }
        const uint32_t next_item = item + gridDim.x * warps;
        if (next_item < f.items) load_index(next_item);
        float acc[kChains] = {0.0f, 0.0f};
        if (kMode == 0 && kXShared) {
            const uint32_t sb = shared_base();
            FastReader fr[kChains];
            uint32_t ra[kChains];
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                fr[c].hi = br[c].hi; fr[c].lo = br[c].lo; fr[c].off = br[c].off; fr[c].next = sb + br[c].next;
                ra[c] = sb + ri_lane[c];
            }
            const uint32_t l1_abs = sb + dec.l1_lane, xs_abs = sb + xs_a;
            auto step = [&](auto offset) {          // one entry of every chain: lookups first, then the rest
                uint32_t top[kChains], val[kChains], len[kChains];
#pragma unroll
                for (int c = 0; c < kChains; ++c) fast_lookup(fr[c], dec.l1_shift, dec.l1_mul, l1_abs, top[c], val[c], len[c]);
                if (kLong) {
#pragma unroll
                    for (int c = 0; c < kChains; ++c)
                        if ((int32_t)len[c] < 0) resolve_long(top[c], dec, f, val[c], len[c]);
                }
#pragma unroll
                for (int c = 0; c < kChains; ++c)
                    fast_consume_sparse<kRow, decltype(offset)::value * kRow>(fr[c], val[c], len[c], ra[c], xs_abs, acc[c]);
            };
            uint32_t s = 0;
            for (; s + 4 <= common; s += 4) {
                step(std::integral_constant<int, 0>());
                step(std::integral_constant<int, 1>());
                step(std::integral_constant<int, 2>());
                step(std::integral_constant<int, 3>());
#pragma unroll
                for (int c = 0; c < kChains; ++c) ra[c] += 4 * kRow;
            }
            for (; s < common; ++s) {
                step(std::integral_constant<int, 0>());
#pragma unroll
                for (int c = 0; c < kChains; ++c) ra[c] += kRow;
            }
#pragma unroll
            for (int c = 0; c < kChains; ++c) {              // the longer chain's remainder
                br[c].hi = fr[c].hi; br[c].lo = fr[c].lo; br[c].off = fr[c].off; br[c].next = fr[c].next - sb;
                uint32_t r = ra[c] - sb;
                for (uint32_t t = common; t < count[c]; ++t) {
                    const float w = decode_value<kLong>(br[c], dec, f);
                    const uint32_t row = kRow == 2 ? lds16(r) : lds32(r);
                    r += kRow;
                    acc[c] = fmaf(ldsf(xs_a + (row << 2)), w, acc[c]);
                }
            }
        } else if (kMode == 0) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                uint32_t r = ri_lane[c];
                for (uint32_t t = 0; t < count[c]; ++t) {
                    const float w = decode_value<kLong>(br[c], dec, f);
                    const uint32_t row = kRow == 2 ? lds16(r) : lds32(r);
                    r += kRow;
                    acc[c] = fmaf(x[(int64_t)row * xs_i], w, acc[c]);
                }
            }
        } else {
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                float* out = aux + cur.pos0[c] + lane_pos;
                for (uint32_t t = 0; t < count[c]; ++t) out[t] = decode_value<kLong>(br[c], dec, f);
            }
        }
        if (kMode == 0) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) acc[c] = warp_sum(acc[c]);
            if (lane == 0) {
                if (cur.whole_column) {
                    y[(int64_t)cur.col * ys_j] = finish_output(f, acc[0] + acc[1], cur.col);
                } else {
#pragma unroll
                    for (int c = 0; c < kChains; ++c)
                        if ((uint32_t)c < cur.segments) aux[cur.first_unit + c] = acc[c];
                }
            }
        }
        __syncwarp();
        item = next_item;
        if (item < f.items) {
            fetch();
            copies_landed();
            __syncwarp();
        }
    }
}

// This lane's sub-segment bit length in segment c of a work item (the copy kept inside the item record).
__device__ __forceinline__ uint32_t load_item_bits(const void* base, uint32_t index, uint32_t c, uint32_t lane) {
    const uint16_t* h = reinterpret_cast<const uint16_t*>(reinterpret_cast<const uint32_t*>(base) +
                                                          (size_t)index * kItemWords + 12 + 16 * c);
    return __ldg(h + lane);
}

// ------------------------------------------------------------------------------------------------
// sHAC, one input vector (Algorithm 2 by segments), the kernel used when x and all staging areas fit in
// shared memory.  A warp takes one work item at a time (up to two segments of one column = two decode
// chains per lane).  Everything an item needs to be located comes in one read of its record; its two
// spans of the stream and two slices of ri are then brought in by four bulk asynchronous copies (TMA,
// issued by one lane, completion on the warp's own mbarrier), x by one more for the block.  Code words
// are decoded three to a window (lookup3); the row of an entry comes from the staged slice of ri and
// x is gathered from shared memory by row.
//   kMode 0: product; 1: debug decode (values written to aux[position in nz]).
// Every mbarrier wait is bounded; if one runs out the data is copied with ordinary loads instead.
// ------------------------------------------------------------------------------------------------
template <int kMode, int kTab, bool kLong, bool kGuard, typename RowT>
__global__ void __launch_bounds__(1024) shac_items_kernel(DevFormat f, TablePlan tp, const float* __restrict__ x,
                                                          int64_t xs_i, float* __restrict__ y, int64_t ys_j,
                                                          float* __restrict__ aux) {
    constexpr int kC = 2;
    constexpr uint32_t kRow = (uint32_t)sizeof(RowT);
    __shared__ DevFormat sf;               // for the rare paths that are calls (decode3_slow)
    allow_dependents();
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
    const uint32_t sb = shared_base();
    const uint32_t xbar = sb, wbar = sb + 16 + 8 * warp;
    // mbarriers first: the fence that publishes them would wait for any load already in flight
    if (threadIdx.x == 0) mbar_init(xbar, 1);
    if (lane == 0) mbar_init(wbar, 1);
    __syncwarp();
    uint32_t item = blockIdx.x + gridDim.x * warp;
    ShacItem info;
    info.segments = 0;
    uint32_t my_bits[kC] = {0, 0};
    // one trip: header and both arrays of lengths (zeros for an absent segment).  Taking the header apart
    // waits for it, so the first record is asked for after everything else that can be in flight by then.
    auto load_index = [&](uint32_t it) {
#pragma unroll
        for (int c = 0; c < kC; ++c) my_bits[c] = load_item_bits(f.unit_info, it, c, lane);
        info = load_item(f.unit_info, it);
    };
    if (threadIdx.x == 0) sf = f;
    // table entries: every warp takes groups of 32 consecutive entries, all its loads in flight at once
    constexpr int kTabAhead = 2;
    const uint32_t entries = f.l1_entries;
    uint2 te[kTabAhead];
#pragma unroll
    for (int i = 0; i < kTabAhead; ++i) {
        const uint32_t idx = (warp + i * warps) * 32 + lane;
        te[i] = idx < entries ? __ldg(f.l1 + idx) : make_uint2(0u, 0u);
    }
    // shared memory: [mbarrier of x, mbarriers of the warps][x][tables][spans: warp, chain][ri slices: warp, chain]
    unsigned char* p = smem + align16(16 + 8 * (size_t)warps);
    float* xs = reinterpret_cast<float*>(p);
    if (kMode == 0) p += align16((size_t)f.n * 4);
    uint2* l1 = reinterpret_cast<uint2*>(p);
    uint2* subt = reinterpret_cast<uint2*>(p + (((size_t)8 * f.l1_entries) << tp.repl_log2));
    p += plan_smem_bytes(f.l1_entries, tp.repl_log2, f.sub_bytes);
    const uint32_t span_bytes = f.max_unit_chunks * 16;
    const uint32_t ri_bytes = kMode == 0 ? ((32u * f.S * kRow + 15u) / 16u + 1u) * 16u : 0u;
    const uint32_t stage_a = smem_off(p) + warp * kC * span_bytes;
    const uint32_t ri_a = smem_off(p) + warps * kC * span_bytes + warp * kC * ri_bytes;
    const uint32_t xs_a = smem_off(xs);
    const RowT* __restrict__ ri = reinterpret_cast<const RowT*>(f.ri);
    const bool bulk = kMode == 0 && tp.x_bulk;
    const uint32_t bulk_bytes = (f.n & ~3u) * 4u;

    // requests the spans and slices of ri of the item whose record is in `info`; pos[c] = bit position of this
    // lane's first code word relative to the staged span of chain c, ri_lane[c] = address of its first row index
    uint32_t pos[kC], ri_lane[kC];
    bool copy_lost = false;
    auto fetch = [&]() {
        uint32_t bytes_total = 0;
        const uint4* src_s[kC]; const uint4* src_r[kC];
        uint32_t n_s[kC], n_r[kC];
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            uint32_t total;
            const uint32_t start = lane_start_bits(my_bits[c], lane, total);
            pos[c] = 0; ri_lane[c] = ri_a; n_s[c] = 0; n_r[c] = 0; src_s[c] = nullptr; src_r[c] = nullptr;
            if ((uint32_t)c < info.segments) {
                const uint64_t first_chunk = info.bit_off[c] >> 7;
                const uint64_t last_word = ((info.bit_off[c] + total) >> 5) + 2;
                n_s[c] = (uint32_t)((last_word >> 2) - first_chunk + 1);
                src_s[c] = reinterpret_cast<const uint4*>(f.stream) + first_chunk;
                pos[c] = start + (uint32_t)(info.bit_off[c] - (first_chunk << 7));
                if (kMode == 0) {
                    const uintptr_t byte0 = reinterpret_cast<uintptr_t>(ri + info.pos0[c]);
                    const uintptr_t chunk0 = byte0 & ~(uintptr_t)15;
                    n_r[c] = (uint32_t)((byte0 + (uintptr_t)info.count[c] * kRow - chunk0 + 15) >> 4);
                    src_r[c] = reinterpret_cast<const uint4*>(chunk0);
                    ri_lane[c] = ri_a + c * ri_bytes + (uint32_t)(byte0 - chunk0) + lane * f.S * kRow;
                }
                bytes_total += 16u * (n_s[c] + n_r[c]);
            }
        }
        if (lane == 0 && bytes_total > 0) {
            mbar_expect_tx(wbar, bytes_total);
#pragma unroll
            for (int c = 0; c < kC; ++c) {
                if (n_s[c]) bulk_copy_g2s(sb + stage_a + c * span_bytes, src_s[c], 16u * n_s[c], wbar);
                if (n_r[c]) bulk_copy_g2s(sb + ri_a + c * ri_bytes, src_r[c], 16u * n_r[c], wbar);
            }
        }
        __syncwarp();
        return bytes_total;
    };
    // the same copies with ordinary loads: only after a wait on the mbarrier has run out
    auto fetch_plain = [&]() {
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            if ((uint32_t)c >= info.segments) continue;
            uint32_t total = 0;
            for (int l = 0; l < 32; ++l) total += __shfl_sync(0xffffffffu, my_bits[c], l);
            const uint64_t first_chunk = info.bit_off[c] >> 7;
            const uint64_t last_word = ((info.bit_off[c] + total) >> 5) + 2;
            const uint32_t ns = (uint32_t)((last_word >> 2) - first_chunk + 1);
            const uint4* src = reinterpret_cast<const uint4*>(f.stream) + first_chunk;
            uint4* dst = reinterpret_cast<uint4*>(smem + stage_a + c * span_bytes);
            for (uint32_t k = lane; k < ns; k += 32) dst[k] = __ldg(src + k);
            if (kMode == 0) {
                const uintptr_t byte0 = reinterpret_cast<uintptr_t>(ri + info.pos0[c]);
                const uintptr_t chunk0 = byte0 & ~(uintptr_t)15;
                const uint32_t nr = (uint32_t)((byte0 + (uintptr_t)info.count[c] * kRow - chunk0 + 15) >> 4);
                const uint4* srcr = reinterpret_cast<const uint4*>(chunk0);
                uint4* dstr = reinterpret_cast<uint4*>(smem + ri_a + c * ri_bytes);
                for (uint32_t k = lane; k < nr; k += 32) dstr[k] = __ldg(srcr + k);
            }
        }
        __syncwarp();
    };

    // everything above (index, spans of the first item, tables) reads the format only; x and the outputs
    // belong to the kernels before this one
    depends_wait();
    if (bulk) {
        if (threadIdx.x == 0 && bulk_bytes > 0) {
            mbar_expect_tx(xbar, bulk_bytes);
            bulk_copy_g2s(sb + xs_a, x, bulk_bytes, xbar);
        }
        for (uint32_t i = (f.n & ~3u) + threadIdx.x; i < f.n; i += blockDim.x) xs[i] = x[i];
    }
    uint32_t pending = 0;
    if (item < f.items) { load_index(item); pending = fetch(); }
    // tables -> shared memory, replicated (see TablePlan)
    Decoder dec;
    {
        const uint32_t repl = 1u << tp.repl_log2;
        auto spread = [&](uint32_t idx0, uint2 v) {
            uint2* dst = l1 + ((size_t)idx0 << tp.repl_log2);
            const uint32_t warp_slots = min(32u, entries - idx0) << tp.repl_log2;
            for (uint32_t s0 = 0; s0 < warp_slots; s0 += 32) {
                const uint32_t src = (s0 + lane) >> tp.repl_log2;
                uint2 w;
                w.x = __shfl_sync(0xffffffffu, v.x, src & 31u);
                w.y = __shfl_sync(0xffffffffu, v.y, src & 31u);
                if (s0 + lane < warp_slots) dst[s0 + lane] = w;
            }
        };
#pragma unroll
        for (int i = 0; i < kTabAhead; ++i) {
            const uint32_t idx0 = (warp + i * warps) * 32;
            if (idx0 < entries) spread(idx0, te[i]);
        }
        for (uint32_t idx0 = (warp + kTabAhead * warps) * 32; idx0 < entries; idx0 += warps * 32) {
            const uint32_t idx = idx0 + lane;
            spread(idx0, idx < entries ? __ldg(f.l1 + idx) : make_uint2(0u, 0u));
        }
        for (uint32_t i = threadIdx.x; i < f.sub_bytes / 8; i += blockDim.x) subt[i] = __ldg(f.sub + i);
        dec.l1_lane = smem_off(l1) + ((threadIdx.x & (repl - 1)) << 3);
        dec.l1_mul = 8u << tp.repl_log2;
        dec.l1_shift = f.tab_kind ? 23 - f.xt_mant : 32 - f.l1_bits;
        dec.bias = f.tab_kind ? (127u + f.xt_row0) << f.xt_mant : 0u;
        dec.xt_low = f.xt_low;
        dec.l1_bits = f.l1_bits;
        dec.sub = smem_off(subt);
    }
    if (kMode == 0 && !bulk) {
#pragma unroll 8
        for (uint32_t i = threadIdx.x; i < f.n; i += blockDim.x) xs[i] = __ldg(x + (int64_t)i * xs_i);
    }
    __syncthreads();                       // tables (and an x copied by ordinary loads) are in place
    if (bulk) {
        const bool landed = bulk_bytes == 0 || mbar_wait_bounded(xbar, 0);
        if (__syncthreads_or(landed ? 0 : 1)) {             // late or lost: copy x the ordinary way
            for (uint32_t i = threadIdx.x; i < f.n; i += blockDim.x) xs[i] = x[i];
            __syncthreads();
        }
    }
    const uint32_t l1_abs = sb + dec.l1_lane - dec.bias * dec.l1_mul, xs_abs = sb + xs_a;
    uint32_t phase = 0;
    while (item < f.items) {
        if (pending) {
            const bool ok = mbar_wait_bounded(wbar, phase);
            if (__any_sync(0xffffffffu, !ok)) { copy_lost = true; fetch_plain(); }
            phase ^= 1u;
        }
        const ShacItem cur = info;
        const uint32_t lane_pos = lane * f.S;
        uint32_t count[kC];
        FastReader fr[kC];
        uint32_t ra[kC];
#pragma unroll
        for (int c = 0; c < kC; ++c) {
            count[c] = ((uint32_t)c < cur.segments && lane_pos < cur.count[c]) ? min(f.S, cur.count[c] - lane_pos) : 0u;
            BitReader br;
            br.init(stage_a + c * span_bytes, pos[c]);
            fr[c].hi = br.hi; fr[c].lo = br.lo; fr[c].off = br.off; fr[c].next = sb + br.next;
            ra[c] = sb + ri_lane[c];
        }
        const uint32_t common = min(count[0], count[1]);
        float acc[kC] = {0.0f, 0.0f};
        float* out[kC];
#pragma unroll
        for (int c = 0; c < kC; ++c) out[c] = aux + cur.pos0[c] + lane_pos;
        // one entry of chain c: value v, the s-th of the lane's sub-segment
        auto apply = [&](int c, uint32_t v, uint32_t s) {
            if (kMode == 0) {
                const uint32_t row = kRow == 2 ? lds16(ra[c] - sb + s * kRow) : lds32(ra[c] - sb + s * kRow);
                acc[c] = fmaf(ldsf(xs_a + (row << 2)), __uint_as_float(v), acc[c]);
            } else {
                out[c][s] = __uint_as_float(v);
            }
        };
        auto triple = [&](int c, uint32_t s) {
            uint32_t v0, v1, v2, tot, flags;
            lookup3<kTab>(fr[c], dec.l1_shift, dec.l1_mul, l1_abs, dec.xt_low, v0, v1, v2, tot, flags);
            if (kGuard || kLong) {
                const bool bad = (kGuard && tot > 32u) || (kLong && (int32_t)flags < 0);
                if (bad) {
                    const Slow3 r = decode3_slow<kTab, kLong>(fr[c].hi, fr[c].lo, fr[c].off, fr[c].next - sb, dec, &sf);
                    fr[c].hi = r.hi; fr[c].lo = r.lo; fr[c].off = r.off; fr[c].next = sb + r.next;
                    v0 = r.v0; v1 = r.v1; v2 = r.v2; tot = 0;
                }
            }
            fast_advance(fr[c], tot);
            apply(c, v0, s); apply(c, v1, s + 1); apply(c, v2, s + 2);
        };
        uint32_t s = 0;
        for (; s + 3 <= common; s += 3) {                         // both chains, three entries each
            triple(0, s);
            triple(1, s);
        }
#pragma unroll
        for (int c = 0; c < kC; ++c) {                            // what one chain has beyond the other, and the ends
            uint32_t t = s;
            for (; t + 3 <= count[c]; t += 3) triple(c, t);
            for (; t < count[c]; ++t) {
                uint32_t top, val, len;
                table_lookup<kTab>(fr[c], dec.l1_shift, dec.l1_mul, l1_abs, dec.xt_low, top, val, len);
                if (kLong && (int32_t)len < 0) resolve_any<kTab>(top, dec, f, val, len);
                fast_advance(fr[c], len);
                apply(c, val, t);
            }
        }
        (void)xs_abs;
        // the record of the next item is requested before the reduction
        const uint32_t next_item = item + gridDim.x * warps;
        __syncwarp();                      // every lane has finished reading the staging areas
        if (next_item < f.items) load_index(next_item);
        if (kMode == 0) {
#pragma unroll
            for (int c = 0; c < kC; ++c) acc[c] = warp_sum(acc[c]);
            if (lane == 0) {
                if (cur.whole_column) {
                    y[(int64_t)cur.col * ys_j] = finish_output(f, acc[0] + acc[1], cur.col);
                } else {
#pragma unroll
                    for (int c = 0; c < kC; ++c)
                        if ((uint32_t)c < cur.segments) aux[cur.first_unit + c] = acc[c];
                }
            }
        }
        item = next_item;
        pending = 0;
        if (item < f.items) pending = fetch();
    }
    (void)copy_lost;
}

// Columns made of several segments (or none): add the per-segment partials in segment order.
//   partial[u*batch + b]; HAC: segments j*G .. j*G+G-1; sHAC: seg_first[j] .. seg_first[j+1]-1.
// Columns with exactly one segment were written by the product kernel itself.
__global__ void finalize_kernel(DevFormat f, bool sparse, const float* __restrict__ partial, uint32_t batch,
                                float* __restrict__ y, int64_t ys_j, int64_t ys_b, uint32_t direct_up_to) {
    allow_dependents();
    depends_wait();
    const uint64_t idx = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (uint64_t)f.m * batch) return;
    const uint32_t j = (uint32_t)(idx / batch), b = (uint32_t)(idx % batch);
    uint32_t u0, u1;
    if (sparse) { u0 = f.seg_first[j]; u1 = f.seg_first[j + 1]; }
    else { u0 = j * f.G; u1 = u0 + f.G; }
    if (u1 - u0 >= 1 && u1 - u0 <= direct_up_to) return;       // written by the product kernel itself
    float s = 0.0f;
    for (uint32_t u = u0; u < u1; ++u) s += partial[(size_t)u * batch + b];
    y[(int64_t)j * ys_j + (int64_t)b * ys_b] = finish_output(f, s, j);
}

// Row splits of the batched HAC kernel: y[j][b] = sum over splits of partial[split][b][j], added in
// split order.  A block handles 32 columns x 32 inputs: it reads along the columns (contiguous in
// the partial sums) and writes along whichever of the two indices is contiguous in y.
__global__ void __launch_bounds__(256) gemm_finalize_kernel(const float* __restrict__ partial, uint32_t splits,
                                                            uint32_t m, uint32_t batch, float* __restrict__ y,
                                                            int64_t ys_j, int64_t ys_b, const float* __restrict__ bias,
                                                            uint32_t relu) {
    __shared__ float tile[32][33];
    allow_dependents();
    depends_wait();
    const uint32_t j0 = blockIdx.x * 32, b0 = blockIdx.y * 32;
    for (uint32_t bb = threadIdx.y; bb < 32; bb += blockDim.y) {
        const uint32_t j = j0 + threadIdx.x, b = b0 + bb;
        float sum = 0.0f;
        if (j < m && b < batch)
            for (uint32_t r = 0; r < splits; ++r) sum += partial[((size_t)r * batch + b) * m + j];
        tile[bb][threadIdx.x] = sum;
    }
    __syncthreads();
    if (ys_b == 1 && ys_j != 1) {
        for (uint32_t jj = threadIdx.y; jj < 32; jj += blockDim.y) {
            const uint32_t j = j0 + jj, b = b0 + threadIdx.x;
            if (j < m && b < batch) y[(int64_t)j * ys_j + b] = finish_output(bias, relu, tile[threadIdx.x][jj], j);
        }
    } else {
        for (uint32_t bb = threadIdx.y; bb < 32; bb += blockDim.y) {
            const uint32_t j = j0 + threadIdx.x, b = b0 + bb;
            if (j < m && b < batch) y[(int64_t)j * ys_j + (int64_t)b * ys_b] = finish_output(bias, relu, tile[bb][threadIdx.x], j);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// HAC, batch of inputs (Algorithm 3 without re-decoding W per input), on the 5th-generation tensor
// cores (tcgen05): Y^T[columns][inputs] = W^T X^T, with W^T as the A operand in tensor memory, X as
// the B operand in shared memory and the accumulators in tensor memory.
//
// A block owns 128 consecutive columns of W (one per tensor-memory lane), a range of sub-segments
// ("tasks": S consecutive rows of every column) and a tile of 64 inputs.  A decode warp serves one
// quarter of the lanes: lane l of the warp decodes column 32q + l, all lanes walking the same rows,
// so the symbols a lane decodes one after the other are consecutive K elements of its own
// accumulator row: they go from registers to tensor memory (tcgen05.st) without a transpose and
// without passing through shared memory.  A lane decodes kGChains tasks at a time, so a stage of 16
// K elements is made of kGChainRows rows of each of them (K need not be contiguous rows of W as long
// as the X tile lists the same rows in the same order).  Four warps per quarter work on different
// tasks at a time; the four warps (one per quarter) that share their tasks form a "slot" with its own
// ring of stages in tensor memory, its own accumulator and its own MMA-issuing thread, so the four
// pipelines never wait for one another (a commit or an mbarrier wait costs the issuing thread
// hundreds of cycles; four threads overlap them).  The epilogue adds the four accumulators.
// Split precision: every weight and every input is written as hi + lo, both rounded to TF32, and
//   D[128][64] += w_hi * x_hi^T + w_hi * x_lo^T + w_lo * x_hi^T
// with three MMAs of N = 64 per 8 K elements.  The error stays near 1e-7 of sum |w x|, well inside the
// output tolerance.
// X is split and tiled once per product by hac_pack_x_kernel, exactly as the tensor core reads it
// ("K-major", no swizzle: four consecutive K elements of one row form a 16-byte unit, 8 rows a
// 128-byte core matrix, successive 8-row groups are kGSbo bytes apart, the two K halves of an MMA
// kGXLbo bytes apart), and comes in with one bulk copy per stage.
// The stream is decoded once per batch tile and never written to global memory.
// ------------------------------------------------------------------------------------------------
constexpr int kBatchSteps = 4;          // sHAC batched kernel: entries decoded per lane per phase
constexpr int kBatchRows = 32 * kBatchSteps;
constexpr int kAccMax = 4;              // sHAC batch tile = 32 * kAcc inputs

__device__ __forceinline__ uint32_t to_tf32(float v) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
    return r;
}

constexpr int kGCols = 128;                         // columns of W per block = accumulator rows
constexpr int kGBatch = 64;                         // inputs per batch tile
constexpr int kGRows = 16;                          // rows of W per tensor-memory stage (two k-steps of 8)
constexpr int kGSlots = 4;                          // decode warps per quarter of the lanes
constexpr int kGStages = 2;                         // tensor-memory stages per slot (each with its own X tile)
constexpr int kGChains = 2;                         // tasks a decode lane works on at a time
constexpr int kGChainRows = kGRows / kGChains;      // rows of each of them in a stage
static_assert(kGChainRows % 4 == 0, "a task fills whole 16-byte units of the X tile");
constexpr int kGDecodeWarps = 4 * kGSlots;
constexpr int kGWarps = kGDecodeWarps + kGSlots;    // plus one MMA-issuing warp per slot
constexpr uint32_t kGDCols = kGSlots * kGBatch;     // one accumulator of 64 columns per slot
constexpr uint32_t kGACols = 2 * kGRows;            // columns of a stage: w_hi | w_lo
constexpr uint32_t kGTmemCols = 512;
static_assert(kGDCols + kGSlots * kGStages * kGACols <= kGTmemCols, "tensor memory holds D and every stage");
constexpr int kGSbo = 128, kGXLbo = 2048, kGXKst = 4096;   // B tile: 128 rows (x_hi of 64 inputs, then x_lo)
constexpr uint32_t kGXLoRows = 8 * kGSbo;           // byte offset of the x_lo rows inside a K half
constexpr uint32_t kGXTileBytes = (kGRows / 8) * kGXKst;
constexpr uint32_t kGMaxSplits = 8;                 // row splits of a product (sizes the partial sums)
constexpr uint32_t kTcWaitTries = 400000;

// shared-memory operand descriptor: K-major, no swizzle
__device__ __forceinline__ uint64_t tc_desc(uint32_t shared_addr, uint32_t lbo_bytes) {
    return (uint64_t)((shared_addr >> 4) & 0x3fffu) | ((uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16) |
           ((uint64_t)((kGSbo >> 4) & 0x3fffu) << 32) | ((uint64_t)1 << 46);
}
// D (tensor memory) (+)= A (tensor memory: lane = row, one column per K element) * B (shared memory)^T
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t mbar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mbar) : "memory");
}
__device__ __forceinline__ bool tc_wait(uint32_t mbar, uint32_t parity) {
    for (uint32_t t = 0; t < kTcWaitTries; ++t) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(mbar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}

// The same wait for a thread that expects to wait long (the MMA-issuing thread, which is ahead of the
// decode warps most of the time): it sleeps between polls so that it does not take issue slots from them.
__device__ __forceinline__ bool tc_wait_idle(uint32_t mbar, uint32_t parity) {
    for (uint32_t t = 0; t < kTcWaitTries; ++t) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(mbar), "r"(parity) : "memory");
        if (done) return true;
        __nanosleep(64);
    }
    return false;
}

// 32 consecutive 32-bit columns of this warp's 32 tensor-memory lanes, one lane per thread.
__device__ __forceinline__ void tmem_ld32(uint32_t (&r)[32], uint32_t taddr) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,"
        "%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
// 16 consecutive columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}

// Work split of the batched HAC kernel.  The tasks (sub-segments) of a column are cut into `row_splits`
// contiguous ranges, one per block; inside a block, slot s and chain c of its `pr`-th round take the
// block's task (pr * kGChains + c) * kGSlots + s.
__host__ __device__ inline uint32_t gemm_split_begin(uint32_t tasks, uint32_t rs, uint32_t row_splits) {
    return (uint32_t)(((uint64_t)tasks * rs) / row_splits);
}
__host__ __device__ inline uint32_t gemm_slot_rounds(uint32_t ntl, uint32_t slot) {
    return slot < ntl ? (ntl - slot + kGChains * kGSlots - 1) / (kGChains * kGSlots) : 0u;
}

// B tiles of hac_gemm_tc_kernel, made once per product.  Tile ((((bt * row_splits + rs) * kGSlots + slot)
// * max_rounds + pr) * cpr + ci) holds what slot `slot` of block (rs, bt) multiplies in chunk ci of its
// round pr: for each of its kGChains tasks, rows ci * kGChainRows .. + kGChainRows - 1 of that task, for the
// 64 inputs of batch tile bt, split into TF32 hi and lo parts and stored exactly as the tile sits in
// shared memory.  Rows past the task or the matrix and inputs past the batch are zero.
// One block of 256 threads per tile, one 16-byte unit of each part per thread.
__global__ void __launch_bounds__(256) hac_pack_x_kernel(DevFormat f, const float* __restrict__ x, int64_t xs_i,
                                                         int64_t xs_b, uint32_t batch, unsigned char* __restrict__ xpack,
                                                         uint32_t tasks, uint32_t row_splits, uint32_t max_rounds,
                                                         uint32_t cpr, uint32_t pack_blocks,
                                                         uint64_t* __restrict__ task_off) {
    allow_dependents();
    depends_wait();                        // x may come from the kernel before; the workspace may still be read by it
    if (blockIdx.x >= pack_blocks) {
        // The remaining blocks turn the offset index into start bits per task, stored [task][column]
        // so that the lanes of a decode warp (consecutive columns, same task) read them coalesced:
        // task_off[t * m + j] = first bit of rows t*S.. of column j; entry `tasks` is the column's end.
        const uint32_t idx = (blockIdx.x - pack_blocks) * blockDim.x + threadIdx.x;     // g * m + j
        if (idx >= f.G * f.m) return;
        const uint32_t g = idx / f.m, j = idx - g * f.m;
        const size_t u = (size_t)j * f.G + g;
        uint64_t at = __ldg(f.seg_bit_off + u);
        const uint4* lens = reinterpret_cast<const uint4*>(f.sub_bits + u * 32);
#pragma unroll
        for (int v4 = 0; v4 < 4; ++v4) {
            const uint4 v = __ldg(lens + v4);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint32_t t = g * 32 + (uint32_t)(8 * v4 + e);
                if (t <= tasks) task_off[(size_t)t * f.m + j] = at;
                if (t < tasks) at += (e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xffffu);
            }
        }
        if (tasks == (g + 1) * 32) task_off[(size_t)tasks * f.m + j] = at;      // the last group is full
        return;
    }
    uint32_t t = blockIdx.x;
    const uint32_t ci = t % cpr; t /= cpr;
    const uint32_t pr = t % max_rounds; t /= max_rounds;
    const uint32_t slot = t % kGSlots; t /= kGSlots;
    const uint32_t rs = t % row_splits, bt = t / row_splits;
    const uint32_t t_begin = gemm_split_begin(tasks, rs, row_splits);
    const uint32_t ntl = gemm_split_begin(tasks, rs + 1, row_splits) - t_begin;
    if (pr >= gemm_slot_rounds(ntl, slot)) return;   // the slot has no such round: the tile is never read
    const uint32_t b = threadIdx.x % kGBatch, kg = threadIdx.x / kGBatch;      // K group of 4 rows
    const uint32_t chain = (kg * 4) / kGChainRows, row0 = (kg * 4) % kGChainRows;
    const uint32_t tl = (pr * kGChains + chain) * kGSlots + slot;
    const uint64_t r0 = (uint64_t)(t_begin + tl) * f.S;
    const uint32_t cnt = tl < ntl ? (uint32_t)min((uint64_t)f.S, (uint64_t)f.n - r0) : 0u;
    const bool b_ok = bt * kGBatch + b < batch;
    const float* xc = x + (int64_t)(bt * kGBatch + b) * xs_b;
    float hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const uint32_t in_task = ci * kGChainRows + row0 + e;
        float v = 0.0f;
        if (b_ok && in_task < cnt) v = __ldg(xc + (int64_t)(r0 + in_task) * xs_i);
        hi[e] = __uint_as_float(to_tf32(v));
        lo[e] = __uint_as_float(to_tf32(v - hi[e]));
    }
    unsigned char* at = xpack + (size_t)blockIdx.x * kGXTileBytes + (kg >> 1) * kGXKst + (kg & 1u) * kGXLbo +
                        (b >> 3) * kGSbo + (b & 7u) * 16;
    *reinterpret_cast<float4*>(at) = make_float4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<float4*>(at + kGXLoRows) = make_float4(lo[0], lo[1], lo[2], lo[3]);
}

// Blocks of the tensor-core kernel whose bounded waits ran out since the library was loaded on this device (their
// outputs are NaN); read by hac_lost_waits.
static __device__ unsigned int g_lost_waits;

// Warps 0..15 decode: warp w serves lane quarter q = w % 4 (columns 32q..32q+31 of the block) in
// slot w / 4.  In every round a lane works on kGChains tasks of its column at once (independent decode
// chains, interleaved instruction by instruction, which hides the latency of the dependent table
// lookups): it copies the stream bytes of those sub-segments to private shared-memory buffers
// (cp.async), and per stage decodes kGChainRows symbols of each, splits them and stores them to its
// tensor-memory lane.  Warp 16 + i holds the MMA-issuing thread of slot i, which also fetches the
// slot's X tiles (one bulk copy per stage).
// mbarriers, per slot and stage: `full` (5 arrivals: one per quarter's warp after its tensor-memory
// stores, one from the thread that requests the X tile, plus the bytes of that bulk copy) and `empty`
// (tcgen05.commit once the MMAs that read the stage have finished).  The X tile of chunk k + 1 shares
// its buffer with chunk k - 1 and is requested once that chunk's MMAs have been committed.
// Every wait is bounded; if one runs out the block marks its outputs NaN and still terminates.
// kSp = 0: HAC (a task is a sub-segment: f.S consecutive rows, one code word per row).  kSp = 2 or 4: sHAC with
// row indices of that many bytes: a task is f.S consecutive rows as well (the caller passes the row-task length
// there), but a column stores code words only for some of them: task_off / task_pos give where the first entry at
// or after the task's first row starts in the stream and in ri, the lane copies that slice of ri next to its span
// of the stream, and a row without an entry contributes a zero to the tile.
template <int kTab, bool kLong, int kSp>
__global__ void __launch_bounds__(kGWarps * 32, 1) hac_gemm_tc_kernel(
    DevFormat f, TablePlan tp, const unsigned char* __restrict__ xpack, uint32_t batch, float* __restrict__ y,
    int64_t ys_j, int64_t ys_b, float* __restrict__ partial, const uint64_t* __restrict__ task_off,
    uint32_t col_blocks, uint32_t row_splits, uint32_t max_rounds, uint32_t slot_bytes, uint32_t nbuf,
    uint32_t cluster_reduce, const uint32_t* __restrict__ task_pos, uint32_t rslot_bytes) {
    allow_dependents();
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // the row splits of a column block are consecutive blocks (one thread-block cluster when cluster_reduce is set)
    const uint32_t rs = blockIdx.x % row_splits;
    const uint32_t rest = blockIdx.x / row_splits;
    const uint32_t cblk = rest % col_blocks, bt = rest / col_blocks;
    const uint32_t tasks = (uint32_t)(((uint64_t)f.n + f.S - 1) / f.S);          // sub-segments of a column
    const uint32_t t_begin = gemm_split_begin(tasks, rs, row_splits);
    const uint32_t ntl = gemm_split_begin(tasks, rs + 1, row_splits) - t_begin;
    const uint32_t cpr = (f.S + kGChainRows - 1) / kGChainRows;                  // chunks (stages) per round
    const uint32_t sb = shared_base();

    // shared memory: [mbarriers; tensor-memory address; lost flag] [tables] [X buffers] [per-lane stream buffers]
    const uint32_t bar_full = sb, bar_empty = sb + 64, bar_done = sb + 128;       // [slot][stage], 8 bytes each
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 136);
    volatile uint32_t* lost_flag = reinterpret_cast<volatile uint32_t*>(smem + 140);
    unsigned char* p = smem + 256;
    if (threadIdx.x == 0) {
        for (uint32_t i = 0; i < kGSlots * kGStages; ++i) { mbar_init(bar_full + 8 * i, 5); mbar_init(bar_empty + 8 * i, 1); }
        mbar_init(bar_done, kGSlots);
        *lost_flag = 0;
    }
    __syncwarp();
    if (warp == kGDecodeWarps) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sb + 136), "r"(kGTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Decode warps: where the sub-segments of the first two rounds start (start bits per task and column,
    // written by hac_pack_x_kernel).
    const uint32_t dq = warp & 3u, dslot = warp >> 2;
    const uint32_t dj = cblk * kGCols + dq * 32 + lane;                       // this lane's column
    const bool dvalid = warp < kGDecodeWarps && dj < f.m;
    const uint32_t rounds = warp < kGDecodeWarps ? gemm_slot_rounds(ntl, dslot) : 0u;
    // first 16-byte chunk of the stream that holds a sub-segment, and (chunks it spans << 7) | bit
    // position of its first code word inside the first chunk
    struct Loc { uint32_t chunk, span, rchunk, rspan, entries; };
    auto locate = [&](uint32_t pr, Loc (&loc)[kGChains]) {
#pragma unroll
        for (int c = 0; c < kGChains; ++c) {
            loc[c].chunk = 0; loc[c].span = 0; loc[c].rchunk = 0; loc[c].rspan = 0; loc[c].entries = 0;
            const uint32_t tl = (pr * kGChains + c) * kGSlots + dslot;
            if (!dvalid || pr >= rounds || tl >= ntl) continue;
            if (kSp) {
                const uint32_t* pa = task_pos + (size_t)(t_begin + tl) * f.m + dj;
                const uint32_t p0 = __ldg(pa), p1 = __ldg(pa + f.m);
                const uint64_t byte0 = (uint64_t)p0 * kSp, byte1 = (uint64_t)p1 * kSp;
                loc[c].entries = p1 - p0;
                loc[c].rchunk = (uint32_t)(byte0 >> 4);
                loc[c].rspan = (p1 > p0 ? (uint32_t)(((byte1 + 15) >> 4) - (byte0 >> 4)) << 7 : 0u) | (uint32_t)(byte0 & 15u);
            }
            const uint64_t* at = task_off + (size_t)(t_begin + tl) * f.m + dj;
            const uint64_t start = __ldg(at);
            const uint32_t mine = (uint32_t)(__ldg(at + f.m) - start);
            const uint64_t first_chunk = start >> 7;
            const uint64_t last_word = ((start + mine) >> 5) + 2;
            loc[c].chunk = (uint32_t)first_chunk;
            loc[c].span = ((uint32_t)((last_word >> 2) - first_chunk + 1) << 7) | (uint32_t)(start - (first_chunk << 7));
        }
    };
    // Tensor memory and barriers need nothing from the kernel before this one (hac_pack_x_kernel), so they
    // are set up while it still runs; its output is read from here on.  The start bits are requested
    // before the tables are staged so that the trips to memory overlap.
    depends_wait();
    Loc loc_cur[kGChains], loc_next[kGChains];
    locate(0, loc_cur);
    locate(1, loc_next);
    const Decoder dec = stage_decoder<true>(f, tp, p);
    p = smem + ((smem_off(p) + 127u) & ~127u);
    const uint32_t xring = smem_off(p);                                        // [slot][stage]
    p += (size_t)kGSlots * kGStages * kGXTileBytes;
    const uint32_t spans = smem_off(p);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;

    if (warp >= kGDecodeWarps) {
        // ---- slot's X tiles in, MMAs out: one lane, chunk after chunk ----
        const uint32_t slot = warp - kGDecodeWarps;
        if (lane == 0) {
            const uint32_t nchunks = gemm_slot_rounds(ntl, slot) * cpr;
            // D f32, A and B tf32, both K-major, M = 128, N = 64
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(kGBatch >> 3) << 17) |
                                   ((uint32_t)(kGCols >> 4) << 24);
            // the slot's tiles are consecutive: chunk k of the slot is chunk k % cpr of its round k / cpr
            const unsigned char* xt = xpack + ((((size_t)bt * row_splits + rs) * kGSlots + slot) * max_rounds) * cpr *
                                                  (size_t)kGXTileBytes;
            const uint32_t xbuf0 = sb + xring + slot * kGStages * kGXTileBytes;
            const uint32_t full0 = bar_full + 8 * slot * kGStages, empty0 = bar_empty + 8 * slot * kGStages;
            const uint32_t d_col = tmem + slot * kGBatch;
            auto fetch_x = [&](uint32_t k) {
                const uint32_t bar = full0 + 8 * (k % kGStages);
                mbar_expect_tx(bar, kGXTileBytes);
                bulk_copy_g2s(xbuf0 + (k % kGStages) * kGXTileBytes, xt + (size_t)k * kGXTileBytes, kGXTileBytes, bar);
            };
            for (uint32_t k = 0; k < kGStages && k < nchunks; ++k) fetch_x(k);
            for (uint32_t k = 0; k < nchunks; ++k) {
                const uint32_t st = k % kGStages;
                // the X tile of chunk k + 1 goes where that of chunk k - 1 was: wait for that chunk's MMAs
                if (k >= 1 && k + 1 < nchunks && k + 1 >= kGStages) {
                    if (!tc_wait(empty0 + 8 * ((k - 1) % kGStages), ((k - 1) / kGStages) & 1u)) *lost_flag = 1;
                    fetch_x(k + 1);
                }
                if (!tc_wait_idle(full0 + 8 * st, (k / kGStages) & 1u)) *lost_flag = 1;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_col = tmem + kGDCols + (slot * kGStages + st) * kGACols;
                const uint64_t b_hi = tc_desc(xbuf0 + st * kGXTileBytes, kGXLbo);
#pragma unroll
                for (int ks = 0; ks < kGRows / 8; ++ks) {
                    const uint64_t bh = b_hi + (uint64_t)(ks * (kGXKst >> 4)), bl = bh + (uint64_t)(kGXLoRows >> 4);
                    tc_mma_ts(d_col, a_col + ks * 8, bh, idesc, (k | (uint32_t)ks) ? 1u : 0u);          // w_hi * x_hi
                    tc_mma_ts(d_col, a_col + ks * 8, bl, idesc, 1u);                                    // w_hi * x_lo
                    tc_mma_ts(d_col, a_col + kGRows + ks * 8, bh, idesc, 1u);                           // w_lo * x_hi
                }
                tc_commit(empty0 + 8 * st);
            }
            tc_commit(bar_done);
        }
        __syncwarp();                        // the other lanes sleep here until the last MMA is issued
    } else {
        // ---- decode -> tensor memory ----
        const uint32_t q = dq, slot = dslot;
        const bool valid = dvalid;
        const bool all_valid = __all_sync(0xffffffffu, valid);
        const uint32_t buf_stride = 32 * slot_bytes;
        // this lane's buffers: [parity][chain], buf_stride apart; the slices of ri (sHAC) lie behind all of them
        const uint32_t my_buf = spans + warp * nbuf * kGChains * buf_stride + lane * slot_bytes;
        const uint32_t rbuf_stride = 32 * rslot_bytes;
        const uint32_t my_rbuf = spans + kGDecodeWarps * nbuf * kGChains * buf_stride + warp * nbuf * kGChains * rbuf_stride +
                                 lane * rslot_bytes;
        const uint32_t l1_abs = sb + dec.l1_lane - dec.bias * dec.l1_mul;
        const uint32_t a_base = tmem + ((q * 32u) << 16) + kGDCols + slot * kGStages * kGACols;
        const uint32_t full0 = bar_full + 8 * slot * kGStages, empty0 = bar_empty + 8 * slot * kGStages;
        // the copies of one round (the located sub-segment of every chain), as one cp.async group
        auto copy_round = [&](const Loc (&loc)[kGChains], uint32_t par) {
            const uint4* stream4 = reinterpret_cast<const uint4*>(f.stream);
#pragma unroll
            for (int c = 0; c < kGChains; ++c) {
                const uint4* src = stream4 + loc[c].chunk;
                const uint32_t dst = sb + my_buf + (par * kGChains + c) * buf_stride, nch = loc[c].span >> 7;
                for (uint32_t i = 0; i < nch; ++i) cp_async16(dst + 16 * i, src + i);
                if (kSp) {
                    const uint4* rsrc = reinterpret_cast<const uint4*>(f.ri) + loc[c].rchunk;
                    const uint32_t rdst = sb + my_rbuf + (par * kGChains + c) * rbuf_stride, rn = loc[c].rspan >> 7;
                    for (uint32_t i = 0; i < rn; ++i) cp_async16(rdst + 16 * i, rsrc + i);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        uint32_t par = 0, k = 0;
        const bool guard = 3u * f.max_len > 32u;       // three code words may not fit one window
        if (rounds > 0) copy_round(loc_cur, 0);
        for (uint32_t pr = 0; pr < rounds; ++pr) {
            const bool more = pr + 1 < rounds;
            if (nbuf == 2 && more) {
                copy_round(loc_next, par ^ 1u);
                asm volatile("cp.async.wait_group 1;" ::: "memory");
            } else {
                asm volatile("cp.async.wait_group 0;" ::: "memory");
            }
            // the index entries of the round after next are in flight while this round is decoded
            Loc loc_after[kGChains];
            locate(pr + 2, loc_after);
            uint32_t bitpos[kGChains];
#pragma unroll
            for (int c = 0; c < kGChains; ++c) bitpos[c] = loc_cur[c].span & 127u;
            FastReader fr[kGChains];
            uint32_t cnt[kGChains];
            uint32_t left[kGChains], nrow[kGChains], rp[kGChains], rowbase[kGChains];    // sHAC: entries left, row of the next, where it is read
            uint32_t full_rows = f.S;                 // rows every chain of the round has
#pragma unroll
            for (int c = 0; c < kGChains; ++c) {
                const uint32_t tl = (pr * kGChains + c) * kGSlots + slot;
                cnt[c] = tl < ntl ? (uint32_t)min((uint64_t)f.S, (uint64_t)f.n - (uint64_t)(t_begin + tl) * f.S) : 0u;
                full_rows = min(full_rows, cnt[c]);
                fr[c].hi = fr[c].lo = fr[c].off = 0; fr[c].next = sb + my_buf;
                left[c] = 0; nrow[c] = 0xffffffffu; rp[c] = 0; rowbase[c] = (t_begin + tl) * f.S;
                if (kSp && valid && cnt[c] > 0 && loc_cur[c].entries > 0) {
                    left[c] = loc_cur[c].entries;
                    rp[c] = my_rbuf + (par * kGChains + c) * rbuf_stride + (loc_cur[c].rspan & 127u);
                    nrow[c] = kSp == 2 ? lds16(rp[c]) : lds32(rp[c]);
                }
                if (valid && cnt[c] > 0) {
                    BitReader br;
                    br.init(my_buf + (par * kGChains + c) * buf_stride, bitpos[c]);
                    fr[c].hi = br.hi; fr[c].lo = br.lo; fr[c].off = br.off; fr[c].next = sb + br.next;
                }
            }
            for (uint32_t r = 0; r < cpr * kGChainRows; r += kGChainRows, ++k) {
                uint32_t hi[kGRows], lo[kGRows];
                // the table entries are {lo, hi | length}: the symbol is ready for the tensor core as it is
                if (kSp) {
                    // sHAC: a row of the tile is the column's next stored entry if that entry lies in this row, else zero
                    // (a variant that looks every row up and only selects was measured: 4 % faster at 60 % zeros, 16 %
                    // slower at 96 %)
#pragma unroll
                    for (int s = 0; s < kGChainRows; ++s) {
#pragma unroll
                        for (int c = 0; c < kGChains; ++c) {
                            uint32_t top = 0, wl = 0, wh = 0;
                            if (nrow[c] == rowbase[c] + r + s) {
                                table_lookup<kTab>(fr[c], dec.l1_shift, dec.l1_mul, l1_abs, dec.xt_low, top, wl, wh);
                                if (kLong && (wh & kSplitLong)) resolve_split_any<kTab>(top, dec, f, wl, wh);
                                fast_consume_value(fr[c], wh & 63u);
                                rp[c] += kSp;
                                nrow[c] = --left[c] ? (kSp == 2 ? lds16(rp[c]) : lds32(rp[c])) : 0xffffffffu;
                            }
                            hi[c * kGChainRows + s] = wh & 0xffffe000u;
                            lo[c * kGChainRows + s] = wl;
                        }
                    }
                } else if (all_valid && r + kGChainRows <= full_rows) {
                    // code words in groups of three (and a last group of two) per window
                    auto one_by_one = [&](int c, int s0, int cntg) {
                        for (int s = s0; s < s0 + cntg; ++s) {
                            uint32_t top, wl1, wh1;
                            table_lookup<kTab>(fr[c], dec.l1_shift, dec.l1_mul, l1_abs, dec.xt_low, top, wl1, wh1);
                            if (kLong && (wh1 & kSplitLong)) resolve_split_any<kTab>(top, dec, f, wl1, wh1);
                            fast_consume_value(fr[c], wh1 & 63u);
                            hi[c * kGChainRows + s] = wh1 & 0xffffe000u;
                            lo[c * kGChainRows + s] = wl1;
                        }
                    };
                    auto group = [&](auto count, int s0) {
                        constexpr int N = decltype(count)::value;
                        uint32_t wl[kGChains][N], wh[kGChains][N], tot[kGChains], flags[kGChains];
#pragma unroll
                        for (int c = 0; c < kGChains; ++c)
                            lookup_group_split<kTab, N>(fr[c], dec.l1_shift, dec.l1_mul, l1_abs, dec.xt_low, wl[c], wh[c], tot[c], flags[c]);
                        bool bad = false;
#pragma unroll
                        for (int c = 0; c < kGChains; ++c) bad = bad || (guard && tot[c] > 32u) || (kLong && flags[c] != 0u);
                        if (bad) {
#pragma unroll
                            for (int c = 0; c < kGChains; ++c) one_by_one(c, s0, N);
                        } else {
#pragma unroll
                            for (int c = 0; c < kGChains; ++c) {
                                fast_consume_value(fr[c], tot[c]);
#pragma unroll
                                for (int e = 0; e < N; ++e) {
                                    hi[c * kGChainRows + s0 + e] = wh[c][e] & 0xffffe000u;
                                    lo[c * kGChainRows + s0 + e] = wl[c][e];
                                }
                            }
                        }
                    };
                    static_assert(kGChainRows == 8, "groups of 3 + 3 + 2 code words");
                    group(std::integral_constant<int, 3>(), 0);
                    group(std::integral_constant<int, 3>(), 3);
                    group(std::integral_constant<int, 2>(), 6);
                } else {
#pragma unroll
                    for (int s = 0; s < kGChainRows; ++s) {
#pragma unroll
                        for (int c = 0; c < kGChains; ++c) {
                            uint32_t top = 0, wl = 0, wh = 0;
                            if (valid && r + s < cnt[c]) {
                                table_lookup<kTab>(fr[c], dec.l1_shift, dec.l1_mul, l1_abs, dec.xt_low, top, wl, wh);
                                if (kLong && (wh & kSplitLong)) resolve_split_any<kTab>(top, dec, f, wl, wh);
                                fast_consume_value(fr[c], wh & 63u);
                            }
                            hi[c * kGChainRows + s] = wh & 0xffffe000u;
                            lo[c * kGChainRows + s] = wl;
                        }
                    }
                }
                const uint32_t st = k % kGStages;
                // the stage is free once the MMAs of its previous use have been committed (one lane polls)
                if (k >= kGStages) {
                    if (lane == 0 && !tc_wait(empty0 + 8 * st, ((k / kGStages) - 1) & 1u)) *lost_flag = 1;
                    __syncwarp();
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                tmem_st16(a_base + st * kGACols, hi);
                tmem_st16(a_base + st * kGACols + kGRows, lo);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(full0 + 8 * st) : "memory");
            }
            if (nbuf == 2) par ^= 1u;
            else if (more) copy_round(loc_next, 0);
#pragma unroll
            for (int c = 0; c < kGChains; ++c) { loc_cur[c] = loc_next[c]; loc_next[c] = loc_after[c]; }
        }
    }
    // ---- epilogue: accumulators -> y ----
    bool lost = false;
    // one lane waits for the last commits; everyone else sleeps in the block barrier below
    if (warp == kGDecodeWarps && lane == 0 && !tc_wait_idle(bar_done, 0)) lost = true;
    const bool any_lost = __syncthreads_or((lost || *lost_flag) ? 1 : 0) != 0;
    if (any_lost && threadIdx.x == 0) atomicAdd(&g_lost_waits, 1u);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp < 4) {
        // lane l of warp q holds column 32q + l; slot s accumulated its tasks in columns 64s..64s+63
        const uint32_t j = cblk * kGCols + warp * 32 + lane;
#pragma unroll 1
        for (uint32_t half = 0; half < 2; ++half) {
            float acc[32];
#pragma unroll
            for (int cc = 0; cc < 32; ++cc) acc[cc] = any_lost ? __uint_as_float(0x7fc00000u) : 0.0f;   // NaN marks a lost wait
            if (!any_lost) {
#pragma unroll 1
                for (uint32_t s = 0; s < kGSlots; ++s) {
                    if (gemm_slot_rounds(ntl, s) == 0) continue;         // that accumulator was never written
                    uint32_t r[32];
                    tmem_ld32(r, tmem + ((warp * 32u) << 16) + s * kGBatch + half * 32);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int cc = 0; cc < 32; ++cc) acc[cc] += __uint_as_float(r[cc]);
                }
            }
            // Stores are made along whichever index is contiguous in memory.  The partial sums are laid
            // out [split][input][column], so lanes (columns) are contiguous there, and so they are in y
            // when y_stride_j is 1; otherwise the 32 x 32 block goes through shared memory (the stream
            // buffers are free by now) and is stored with the lanes along the inputs.
            const uint32_t b0 = bt * kGBatch + half * 32;
            if (row_splits > 1 && cluster_reduce) {
                // this block's 128 x 64 tile of sums goes to its shared memory, in the orientation of y
                float* tile = reinterpret_cast<float*>(smem + spans);
                if (ys_b == 1 && ys_j != 1) {
#pragma unroll
                    for (int cc = 0; cc < 32; ++cc) tile[(warp * 32 + lane) * (kGBatch + 1) + half * 32 + cc] = acc[cc];
                } else {
#pragma unroll
                    for (int cc = 0; cc < 32; ++cc) tile[(half * 32 + cc) * kGCols + warp * 32 + lane] = acc[cc];
                }
            } else if (row_splits > 1) {
                if (j < f.m) {
#pragma unroll
                    for (int cc = 0; cc < 32; ++cc)
                        if (b0 + cc < batch) partial[((size_t)rs * batch + b0 + cc) * f.m + j] = acc[cc];
                }
            } else if (ys_j == 1) {
                if (j < f.m) {
#pragma unroll
                    for (int cc = 0; cc < 32; ++cc)
                        if (b0 + cc < batch) y[(int64_t)j + (int64_t)(b0 + cc) * ys_b] = finish_output(f, acc[cc], j);
                }
            } else {
                float* tile = reinterpret_cast<float*>(smem + spans) + warp * (32 * 33);
                __syncwarp();
#pragma unroll
                for (int cc = 0; cc < 32; ++cc) tile[cc * 33 + lane] = acc[cc];
                __syncwarp();
                const uint32_t jw = cblk * kGCols + warp * 32;
                if (b0 + lane < batch) {
                    float* yb = y + (int64_t)(b0 + lane) * ys_b;
                    const uint32_t jn = min(32u, f.m > jw ? f.m - jw : 0u);
                    for (uint32_t jj = 0; jj < jn; ++jj) yb[(int64_t)(jw + jj) * ys_j] = finish_output(f, tile[lane * 33 + jj], jw + jj);
                }
            }
        }
    }
    if (row_splits > 1 && cluster_reduce) {
        // The blocks of the cluster hold the row splits of the same 128 columns: each adds, in split order, its
        // share of the outputs from everybody's tile (distributed shared memory) and writes it to y.
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        const uint32_t tile_a = sb + spans;
        auto remote = [&](uint32_t byte_off, uint32_t rank) {
            uint32_t a;
            float v;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(tile_a + byte_off), "r"(rank));
            asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(a) : "memory");
            return v;
        };
        if (ys_b == 1 && ys_j != 1) {               // y is [column][input]: a share of the columns, inputs fastest
            const uint32_t j0 = kGCols * rs / row_splits, j1 = kGCols * (rs + 1) / row_splits;
            for (uint32_t idx = threadIdx.x; idx < (j1 - j0) * kGBatch; idx += blockDim.x) {
                const uint32_t jl = j0 + idx / kGBatch, b = idx % kGBatch;
                float sum = 0.0f;
                for (uint32_t r = 0; r < row_splits; ++r) sum += remote((jl * (kGBatch + 1) + b) * 4u, r);
                const uint32_t j = cblk * kGCols + jl, bb = bt * kGBatch + b;
                if (j < f.m && bb < batch) y[(int64_t)j * ys_j + bb] = finish_output(f, sum, j);
            }
        } else {                                     // a share of the inputs, columns fastest
            const uint32_t b0 = kGBatch * rs / row_splits, b1 = kGBatch * (rs + 1) / row_splits;
            for (uint32_t idx = threadIdx.x; idx < (b1 - b0) * kGCols; idx += blockDim.x) {
                const uint32_t b = b0 + idx / kGCols, jl = idx % kGCols;
                float sum = 0.0f;
                for (uint32_t r = 0; r < row_splits; ++r) sum += remote((b * kGCols + jl) * 4u, r);
                const uint32_t j = cblk * kGCols + jl, bb = bt * kGBatch + b;
                if (j < f.m && bb < batch) y[(int64_t)j * ys_j + (int64_t)bb * ys_b] = finish_output(f, sum, j);
            }
        }
        // nobody leaves while its tile may still be read
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == kGDecodeWarps) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kGTmemCols) : "memory");
}

// ------------------------------------------------------------------------------------------------
// sHAC, batch of inputs.  One warp per segment: lanes decode kBatchSteps entries each into a small
// shared tile of (value, row) pairs, then the warp walks the tile with lanes spread over the
// inputs, gathering the rows of X (stored [n][batch] for coalesced access).  With 16 inputs or fewer
// the lanes are split into groups of `narrow` (a power of two that holds the batch): every group
// takes its own entry of the tile, and the groups' sums are added with shuffles at the end.
// ------------------------------------------------------------------------------------------------
template <int kAcc, typename RowT>
__global__ void __launch_bounds__(1024) shac_batch_kernel(DevFormat f, TablePlan tp, const float* __restrict__ x,
                                                          int64_t xs_i, int64_t xs_b, uint32_t batch,
                                                          float* __restrict__ y, int64_t ys_j, int64_t ys_b,
                                                          float* __restrict__ partial, uint32_t narrow) {
    unsigned char* p = smem;
    const Decoder dec = stage_decoder(f, tp, p);
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
    constexpr uint32_t kTile = 32 * kAcc;
    float* wv_all = reinterpret_cast<float*>(p);
    p += align16((size_t)warps * kBatchRows * 4);
    uint32_t* wr_all = reinterpret_cast<uint32_t*>(p);
    p += align16((size_t)warps * kBatchRows * 4);
    uint4* stage = reinterpret_cast<uint4*>(p) + (size_t)warp * f.max_unit_chunks;
    float* wv = wv_all + warp * kBatchRows;
    uint32_t* wr = wr_all + warp * kBatchRows;
    const uint32_t stage_a = smem_off(stage);
    __syncthreads();
    const RowT* __restrict__ ri = reinterpret_cast<const RowT*>(f.ri);
    const uint32_t batch_tiles = (batch + kTile - 1) / kTile;
    const uint64_t items = (uint64_t)f.units * batch_tiles;

    for (uint64_t item = (uint64_t)blockIdx.x * warps + warp; item < items; item += (uint64_t)gridDim.x * warps) {
        const uint32_t u = (uint32_t)(item / batch_tiles);
        const uint32_t b0 = (uint32_t)(item % batch_tiles) * kTile;
        const uint32_t j = f.seg_col[u];
        const uint32_t first = f.seg_first[j];
        const uint32_t g = u - first;
        const uint32_t col_end = f.cb[j + 1];
        const uint32_t my_bits = f.sub_bits[(size_t)u * 32 + lane];
        uint32_t total;
        const uint32_t start = lane_start_bits(my_bits, lane, total);
        const uint32_t base = stage_span(f, f.seg_bit_off[u], total, stage, lane);
        copies_landed();
        __syncwarp();
        const uint32_t seg_pos0 = f.cb[j] + g * 32 * f.S;
        const uint32_t pos0 = seg_pos0 + lane * f.S;
        const uint32_t count = pos0 < col_end ? min(f.S, col_end - pos0) : 0u;
        const uint32_t seg_rows = min(f.S, col_end - seg_pos0);
        BitReader br;
        br.init(stage_a, base + start);
        float acc[kAcc];
#pragma unroll
        for (int a = 0; a < kAcc; ++a) acc[a] = 0.0f;
        for (uint32_t s0 = 0; s0 < seg_rows; s0 += kBatchSteps) {
#pragma unroll
            for (int s = 0; s < kBatchSteps; ++s) {
                float v = 0.0f;
                uint32_t row = 0;
                if (s0 + s < count) {
                    v = decode_value<true>(br, dec, f);
                    row = ri[pos0 + s0 + s];
                }
                wv[lane * kBatchSteps + s] = v;
                wr[lane * kBatchSteps + s] = row;
            }
            __syncwarp();
            if (kAcc == 1 && narrow) {
                // few inputs: `narrow` lanes per entry, 32 / narrow entries at a time
                const uint32_t e = lane / narrow, b = lane % narrow;
                if (b < batch) {
#pragma unroll 4
                    for (uint32_t r = e; r < kBatchRows; r += 32 / narrow)
                        acc[0] = fmaf(wv[r], x[(int64_t)wr[r] * xs_i + (int64_t)b * xs_b], acc[0]);
                }
            } else {
#pragma unroll 4
                for (uint32_t r = 0; r < kBatchRows; ++r) {
                    const float v = wv[r];
                    const float* xr = x + (int64_t)wr[r] * xs_i;
#pragma unroll
                    for (int a = 0; a < kAcc; ++a) {
                        const uint32_t b = b0 + a * 32 + lane;
                        if (b < batch) acc[a] = fmaf(v, xr[(int64_t)b * xs_b], acc[a]);
                    }
                }
            }
            __syncwarp();
        }
        if (kAcc == 1 && narrow) {               // add the entry groups; lanes 0 .. narrow-1 hold the sums
            for (uint32_t d = narrow; d < 32; d <<= 1) acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], d);
        }
        const bool writer = !(kAcc == 1 && narrow) || lane < narrow;
        const bool single = (f.seg_first[j + 1] - first) == 1;
#pragma unroll
        for (int a = 0; a < kAcc; ++a) {
            const uint32_t b = b0 + a * 32 + lane;
            if (writer && b < batch) {
                if (single) y[(int64_t)j * ys_j + (int64_t)b * ys_b] = finish_output(f, acc[a], j);
                else partial[(size_t)u * batch + b] = acc[a];
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// sHAC, batch of inputs, rows of X staged in shared memory.  The row tasks of the format (f.S consecutive rows
// here; task_off / task_pos give, per task and column, where the column's first stored entry at or after the
// task's first row starts in the stream and in ri) cut every column into cells.  A block owns kRbCols
// consecutive columns, a range of tasks (the row split) and a tile of 32 * kIn inputs.  It walks its tasks in
// groups of `group` tasks: the group's rows of X for its inputs are brought into shared memory (coalesced
// 16-byte asynchronous copies), then every warp works off the cells of its eight columns, 32 cells at a time
// (lane l: column l % 8, task l / 8 of the pass): every lane decodes one entry of its cell straight from global
// memory (a cell is a handful of code words), and for every entry so decoded the whole warp multiplies its value
// with the entry's row of X, lane l holding inputs l * kIn .. + kIn - 1 of each of the eight column sums.  X is
// thus read from memory once per block of 256 columns, not once per stored entry.  Sums of a row split go to
// partial[split][column][input] for rowblock_finalize_kernel; without a split y is written directly.
// ------------------------------------------------------------------------------------------------
// A warp has kWC columns (8, or 4 when the tile is 128 inputs wide and eight columns' sums would not fit the registers) and
// 32 / kWC tasks per pass, so 32 cells either way; a column collects up to kRbChunk entries of each of those tasks.
constexpr uint32_t kRbWarps = 32, kRbChunk = 4;
constexpr size_t kRbListBytes = (size_t)kRbWarps * 32 * kRbChunk * 8;

template <int kIn, int kWC, typename RowT>
__global__ void __launch_bounds__(kRbWarps * 32, 1)
shac_rowblock_kernel(DevFormat f, TablePlan tp, const float* __restrict__ x, int64_t xs_i, uint32_t batch,
                     float* __restrict__ y, int64_t ys_j, int64_t ys_b, float* __restrict__ partial,
                     const uint64_t* __restrict__ task_off, const uint32_t* __restrict__ task_pos, uint32_t tasks,
                     uint32_t row_splits, uint32_t col_blocks, uint32_t nbuf, uint32_t x_aligned, uint32_t group) {
    constexpr uint32_t kTileB = 32 * kIn;
    constexpr uint32_t kPassTasks = 32 / kWC, kListLen = kPassTasks * kRbChunk;
    constexpr uint32_t kTaskBits = kWC == 8 ? 0x01010101u : 0x11111111u;      // ballot bits of one column: one per task of the pass
    allow_dependents();
    unsigned char* p = smem;
    const Decoder dec = stage_decoder(f, tp, p);
    // decoded entries of the pass at hand, per warp and column: kRbChunk steps x four tasks of {value, row in the group}
    uint2* lists = reinterpret_cast<uint2*>(smem + ((smem_off(p) + 15u) & ~15u));
    float* xs = reinterpret_cast<float*>(lists + (size_t)kRbWarps * kWC * kListLen);      // [nbuf][group * T][kTileB]
    const uint32_t T = f.S, group_rows = group * T;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cblk = blockIdx.x % col_blocks, rs = blockIdx.x / col_blocks;
    const uint32_t b0 = blockIdx.y * kTileB;
    const uint32_t t_begin = gemm_split_begin(tasks, rs, row_splits), t_end = gemm_split_begin(tasks, rs + 1, row_splits);
    const uint32_t jw = cblk * (kRbWarps * kWC) + warp * kWC;
    const uint32_t jc = jw + (lane & (kWC - 1u));
    const RowT* __restrict__ ri = reinterpret_cast<const RowT*>(f.ri);
    float acc[kWC][kIn];
#pragma unroll
    for (int c = 0; c < (int)kWC; ++c)
#pragma unroll
        for (int i = 0; i < kIn; ++i) acc[c][i] = 0.0f;

    // where this lane's cell (its column, task t) starts, and how many entries it holds; t_hi bounds the group
    auto cell = [&](uint32_t t, uint32_t t_hi, uint64_t& bit, uint32_t& p0, uint32_t& cnt) {
        bit = 0; p0 = 0; cnt = 0;
        if (jc < f.m && t < t_hi) {
            const size_t i = (size_t)t * f.m + jc;
            bit = __ldg(task_off + i);
            p0 = __ldg(task_pos + i);
            cnt = __ldg(task_pos + i + f.m) - p0;
        }
    };
    // rows [r0, r0 + nrows) of X for this block's inputs -> shared memory; rows past the matrix and inputs past the
    // batch are zero
    auto stage_x = [&](uint32_t r0, uint32_t nrows, uint32_t buf) {
        float* dst0 = xs + (size_t)buf * group_rows * kTileB;
        constexpr uint32_t kQ = kTileB / 4;
        for (uint32_t idx = threadIdx.x; idx < nrows * kQ; idx += blockDim.x) {
            const uint32_t r = idx / kQ, q = idx % kQ;
            float* dst = dst0 + r * kTileB + 4 * q;
            const uint32_t b = b0 + 4 * q;
            if (r0 + r < f.n && x_aligned && b + 3 < batch) {
                cp_async16((uint32_t)__cvta_generic_to_shared(dst), x + (int64_t)(r0 + r) * xs_i + b);
            } else {
                float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                if (r0 + r < f.n) {
                    const float* src = x + (int64_t)(r0 + r) * xs_i;
                    if (b < batch) v.x = __ldg(src + b);
                    if (b + 1 < batch) v.y = __ldg(src + b + 1);
                    if (b + 2 < batch) v.z = __ldg(src + b + 2);
                    if (b + 3 < batch) v.w = __ldg(src + b + 3);
                }
                *reinterpret_cast<float4*>(dst) = v;
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    auto group_tasks = [&](uint32_t gt) { return min(group, t_end - gt); };

    uint64_t bit_n;
    uint32_t p0_n, cnt_n;
    cell(t_begin + (lane / kWC), min(t_begin + group, t_end), bit_n, p0_n, cnt_n);
    depends_wait();                               // x and the partial sums belong to the kernels before this one
    if (t_begin < t_end) stage_x(t_begin * T, group_tasks(t_begin) * T, 0);
    uint32_t gi = 0;
    for (uint32_t gt = t_begin; gt < t_end; gt += group, ++gi) {
        const uint32_t buf = nbuf == 2 ? (gi & 1u) : 0u;
        const uint32_t g_hi = gt + group_tasks(gt);
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();                          // this group's rows have landed; everyone has left the group before
        if (nbuf == 2 && g_hi < t_end) stage_x(g_hi * T, group_tasks(g_hi) * T, buf ^ 1u);     // lands while this group is worked off
        const float* xb = xs + (size_t)buf * group_rows * kTileB + lane * kIn;
        const uint32_t row0 = gt * T;
        for (uint32_t tp0 = gt; tp0 < g_hi; tp0 += kPassTasks) {               // a pass: 32 cells
            uint64_t bit = bit_n;
            const uint32_t p0 = p0_n, cnt = cnt_n;
            // the cells of the next pass (or of the next group's first pass) are requested now
            if (tp0 + kPassTasks < g_hi) cell(tp0 + kPassTasks + (lane / kWC), g_hi, bit_n, p0_n, cnt_n);
            else cell(g_hi + (lane / kWC), min(g_hi + group, t_end), bit_n, p0_n, cnt_n);
            uint32_t maxc = cnt;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) maxc = max(maxc, __shfl_xor_sync(0xffffffffu, maxc, o));
            if (kIn == 4) {
                // 128 inputs: the eight columns' sums leave no registers for the lists' bookkeeping; every decoded entry is
                // handed to the warp by shuffle instead
                for (uint32_t e = 0; e < maxc; ++e) {
                    float v = 0.0f;
                    uint32_t rr = 0;
                    const bool have = e < cnt;
                    if (have) {
                        const uint32_t* w = f.stream + (bit >> 5);
                        const uint32_t top = __funnelshift_l(__ldg(w + 1), __ldg(w), (uint32_t)bit & 31u);
                        uint2 en = lds64(dec.l1_lane + (top >> dec.l1_shift) * dec.l1_mul);
                        if ((int32_t)en.y < 0) {
                            const uint32_t q = (top << dec.l1_bits) >> (32 - (en.y & 31u));
                            en = lds64(dec.sub + en.x + (q << 3));
                            if (en.y == 0)
                                en = decode_long(top, f.lut, f.lut_bits, f.rank_value, f.limit, f.first_left, f.rank_base, f.max_len);
                        }
                        bit += en.y;
                        v = __uint_as_float(en.x);
                        rr = min((uint32_t)ri[p0 + e] - row0, group_rows - 1);
                    }
                    const uint32_t mask = __ballot_sync(0xffffffffu, have);
                    // column after column (the sums of a column are named registers), the up to four tasks of a column by set bit
    #pragma unroll
                    for (int c = 0; c < (int)kWC; ++c) {
                        uint32_t mc = (mask >> c) & kTaskBits;
                        while (mc) {
                            const int src = __ffs((int)mc) - 1 + c;
                            mc &= mc - 1;
                            const float vc = __shfl_sync(0xffffffffu, v, src);
                            const uint32_t rc = __shfl_sync(0xffffffffu, rr, src);
                            const float* xr = xb + rc * kTileB;
                            if (kIn == 4) {
                                const float4 xv = *reinterpret_cast<const float4*>(xr);
                                acc[c][0] = fmaf(vc, xv.x, acc[c][0]);
                                acc[c][1 % kIn] = fmaf(vc, xv.y, acc[c][1 % kIn]);
                                acc[c][2 % kIn] = fmaf(vc, xv.z, acc[c][2 % kIn]);
                                acc[c][3 % kIn] = fmaf(vc, xv.w, acc[c][3 % kIn]);
                            } else if (kIn == 2) {
                                const float2 xv = *reinterpret_cast<const float2*>(xr);
                                acc[c][0] = fmaf(vc, xv.x, acc[c][0]);
                                acc[c][1 % kIn] = fmaf(vc, xv.y, acc[c][1 % kIn]);
                            } else {
                                acc[c][0] = fmaf(vc, xr[0], acc[c][0]);
                            }
                        }
                    }
                }
            } else {
                uint2* mylist = lists + ((size_t)warp * kWC + (lane & (kWC - 1u))) * kListLen;
                const uint32_t below = (1u << (kWC * (lane / kWC))) - 1u;         // the tasks of my column that come before mine
                for (uint32_t e0 = 0; e0 < maxc; e0 += kRbChunk) {
                    // decode: every lane one entry of its cell per step, appended to its column's list in (step, task) order
                    uint32_t mine = 0;                                           // entries my column has collected (same in its four lanes)
    #pragma unroll 1
                    for (uint32_t de = 0; de < kRbChunk; ++de) {
                        const uint32_t e = e0 + de;
                        const bool have = e < cnt;
                        float v = 0.0f;
                        uint32_t rr = 0;
                        if (have) {
                            const uint32_t* w = f.stream + (bit >> 5);
                            const uint32_t top = __funnelshift_l(__ldg(w + 1), __ldg(w), (uint32_t)bit & 31u);
                            uint2 en = lds64(dec.l1_lane + (top >> dec.l1_shift) * dec.l1_mul);
                            if ((int32_t)en.y < 0) {
                                const uint32_t q = (top << dec.l1_bits) >> (32 - (en.y & 31u));
                                en = lds64(dec.sub + en.x + (q << 3));
                                if (en.y == 0)
                                    en = decode_long(top, f.lut, f.lut_bits, f.rank_value, f.limit, f.first_left, f.rank_base, f.max_len);
                            }
                            bit += en.y;
                            v = __uint_as_float(en.x);
                            rr = min((uint32_t)ri[p0 + e] - row0, group_rows - 1);
                        }
                        const uint32_t mc = (__ballot_sync(0xffffffffu, have) >> (lane & (kWC - 1u))) & kTaskBits;
                        if (have) mylist[mine + __popc(mc & below)] = make_uint2(__float_as_uint(v), rr);
                        mine += __popc(mc);
                    }
                    __syncwarp();
                    // multiply: column after column (the sums of a column are named registers), every lane its inputs
    #pragma unroll
                    for (int c = 0; c < (int)kWC; ++c) {
                        const uint32_t nc = __shfl_sync(0xffffffffu, mine, c);
                        const uint2* lc = lists + ((size_t)warp * kWC + c) * kListLen;
                        for (uint32_t i = 0; i < nc; ++i) {
                            const uint2 en = lc[i];
                            const float vc = __uint_as_float(en.x);
                            const float* xr = xb + en.y * kTileB;
                            if (kIn == 4) {
                                const float4 xv = *reinterpret_cast<const float4*>(xr);
                                acc[c][0] = fmaf(vc, xv.x, acc[c][0]);
                                acc[c][1 % kIn] = fmaf(vc, xv.y, acc[c][1 % kIn]);
                                acc[c][2 % kIn] = fmaf(vc, xv.z, acc[c][2 % kIn]);
                                acc[c][3 % kIn] = fmaf(vc, xv.w, acc[c][3 % kIn]);
                            } else if (kIn == 2) {
                                const float2 xv = *reinterpret_cast<const float2*>(xr);
                                acc[c][0] = fmaf(vc, xv.x, acc[c][0]);
                                acc[c][1 % kIn] = fmaf(vc, xv.y, acc[c][1 % kIn]);
                            } else {
                                acc[c][0] = fmaf(vc, xr[0], acc[c][0]);
                            }
                        }
                    }
                    __syncwarp();
                }
            }
        }
        if (nbuf == 1) {
            __syncthreads();                      // everyone is done with the rows before they are replaced
            if (g_hi < t_end) stage_x(g_hi * T, group_tasks(g_hi) * T, 0);
        }
    }
    // inputs of a lane are consecutive, so a warp writes kTileB consecutive inputs of one column at a time
#pragma unroll
    for (int c = 0; c < (int)kWC; ++c) {
        const uint32_t j = jw + c;
        if (j >= f.m) continue;
#pragma unroll
        for (int i = 0; i < kIn; ++i) {
            const uint32_t b = b0 + lane * kIn + i;
            if (b >= batch) continue;
            if (row_splits == 1) y[(int64_t)j * ys_j + (int64_t)b * ys_b] = finish_output(f, acc[c][i], j);
            else partial[((size_t)rs * f.m + j) * batch + b] = acc[c][i];
        }
    }
}

// y[j][b] = sum over the row splits of partial[split][j][b], added in split order (see shac_rowblock_kernel).
__global__ void __launch_bounds__(256) rowblock_finalize_kernel(const float* __restrict__ partial, uint32_t splits, uint32_t m,
                                                                uint32_t batch, float* __restrict__ y, int64_t ys_j,
                                                                int64_t ys_b, const float* __restrict__ bias, uint32_t relu) {
    allow_dependents();
    depends_wait();
    const uint64_t total = (uint64_t)m * batch;
    for (uint64_t idx = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (uint64_t)gridDim.x * blockDim.x) {
        const uint32_t j = (uint32_t)(idx / batch), b = (uint32_t)(idx % batch);
        float sum = 0.0f;
        for (uint32_t r = 0; r < splits; ++r) sum += partial[(size_t)r * total + idx];
        y[(int64_t)j * ys_j + (int64_t)b * ys_b] = finish_output(bias, relu, sum, j);
    }
}

// X[batch][n] -> Xt[n][batch] (host-input path only).
__global__ void transpose_kernel(const float* __restrict__ in, float* __restrict__ out, uint32_t rows,
                                 uint32_t cols) {
    __shared__ float tile[32][33];
    const uint32_t c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    for (uint32_t r = threadIdx.y; r < 32; r += blockDim.y)
        if (r0 + r < rows && c0 + threadIdx.x < cols) tile[r][threadIdx.x] = in[(size_t)(r0 + r) * cols + c0 + threadIdx.x];
    __syncthreads();
    for (uint32_t c = threadIdx.y; c < 32; c += blockDim.y)
        if (c0 + c < cols && r0 + threadIdx.x < rows) out[(size_t)(c0 + c) * rows + r0 + threadIdx.x] = tile[threadIdx.x][c];
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
void set_last_cuda_error(const std::string& text) { g_last_cuda_error = text; }

struct DeviceInfo {
    int sms = 0;
    int max_smem_optin = 0;
    bool ok = false;
};

static int device_info(DeviceInfo& d) {
    static thread_local DeviceInfo cache[64];
    int dev = 0;
    HAC_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && cache[dev].ok) { d = cache[dev]; return HAC_OK; }
    HAC_CUDA(cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev));
    HAC_CUDA(cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    d.ok = true;
    if (dev >= 0 && dev < 64) cache[dev] = d;
    return HAC_OK;
}

static int env_int(const char* name, int fallback) {
    const char* v = std::getenv(name);
    return v && *v ? std::atoi(v) : fallback;
}

// Diagnostic switches (environment, read once when the first product is launched; see hac.h).
struct Tune {
    int pdl;            // HAC_B200_PDL=0: launch without programmatic stream serialization
    int rows_kernel;    // HAC_B200_ROWS=0: single-input HAC always through the shared-memory-x kernel
    int rows_warps;     // HAC_B200_ROWS_WARPS=n: warps per block of the rows-in-registers kernel (0 = chosen by the library)
    int zero_runs;      // HAC_B200_ZERO_RUNS=0: never use the zero-run table
    int xt;             // HAC_B200_XT=0: never use the magnitude table
    int prefetch;       // HAC_B200_PREFETCH=1: the rows-in-registers kernel asks for its share of the stream into L2 at its start
                        // (measured slightly slower: the requests compete with the index entries; off by default)
    int rows_chains;    // HAC_B200_ROWS_CHAINS=2|3: decode chains per lane of that kernel (0 = chosen by the library)
    int items_kernel;   // HAC_B200_ITEMS=0: single-input sHAC always through the older kernel
    int shac_tc;        // HAC_B200_SHAC_TC=0: batched sHAC never on the tensor cores; 2: always (1 = chosen by estimated cost)
    int vec_warps;      // HAC_B200_VEC_WARPS=n: warps per block of the shared-memory-x kernels (0 = chosen by the library)
    int vec_group;      // HAC_B200_VEC_GROUP=0: the shared-memory-x HAC kernel decodes one code word per lookup
    int gemm_cluster;   // HAC_B200_GEMM_CLUSTER=0: batched HAC adds its row splits in a finishing kernel, not in a cluster
    int shac_rows_group;// HAC_B200_SHAC_ROWS_GROUP=n: row tasks per staged group of that kernel, one buffer (0 = chosen by the library)
    int shac_rows;      // HAC_B200_SHAC_ROWS=0: batched sHAC never through the kernel that stages rows of X; 2: whenever it can
                        // (1 = chosen by estimated cost)
};
static const Tune& tune() {
    static const Tune t = {env_int("HAC_B200_PDL", 1), env_int("HAC_B200_ROWS", 1), env_int("HAC_B200_ROWS_WARPS", 0),
                           env_int("HAC_B200_ZERO_RUNS", 1), env_int("HAC_B200_XT", 1), env_int("HAC_B200_PREFETCH", 0), env_int("HAC_B200_ROWS_CHAINS", 0), env_int("HAC_B200_ITEMS", 1), env_int("HAC_B200_SHAC_TC", 1), env_int("HAC_B200_VEC_WARPS", 0), env_int("HAC_B200_VEC_GROUP", 1), env_int("HAC_B200_GEMM_CLUSTER", 1), env_int("HAC_B200_SHAC_ROWS_GROUP", 0), env_int("HAC_B200_SHAC_ROWS", 1)};
    return t;
}

static DevFormat dev_format(const Format& f) {
    DevFormat d{};
    d.stream = f.dev.stream; d.lut = f.dev.lut; d.rank_value = f.dev.rank_value;
    d.l1 = reinterpret_cast<const uint2*>(f.dev.l1); d.sub = reinterpret_cast<const uint2*>(f.dev.sub);
    d.l1_bits = (uint32_t)f.tables.l1_bits; d.sub_bytes = (uint32_t)(f.tables.sub.size() * 4);
    d.l1_entries = 1u << d.l1_bits;
    d.items = (uint32_t)(f.item_info.size() / kItemWords);
    d.limit = f.dev.limit; d.first_left = f.dev.first_left; d.rank_base = f.dev.rank_base;
    d.seg_bit_off = f.dev.seg_bit_off; d.sub_bits = f.dev.sub_bits; d.seg_col = f.dev.seg_col;
    d.seg_first = f.dev.seg_first; d.ri = f.dev.ri; d.cb = f.dev.cb; d.unit_info = f.dev.unit_info;
    d.n = (uint32_t)f.n; d.m = (uint32_t)f.m; d.units = (uint32_t)f.seg_bit_off.size();
    d.G = f.G ? f.G : 1; d.S = f.S; d.k_eff = (uint32_t)f.codebook.size();
    d.lut_bits = (uint32_t)f.tables.lut_bits; d.max_len = f.max_len; d.ri_bits = f.ri_bits;
    d.max_unit_chunks = f.max_unit_chunks;
    d.max_sub_chunks = f.max_sub_chunks;
    d.tab_kind = 0;
    d.epi_bias = f.epi_bias; d.epi_relu = f.epi_relu;
    return d;
}

// The same with the magnitude table as first-level table, when the format has one that resolves more
// symbols than the prefix table.
static bool wants_xt(const Format& f) { return f.tables.use_xt && tune().xt != 0; }
static DevFormat dev_format_xt(const Format& f) {
    DevFormat d = dev_format(f);
    if (wants_xt(f)) {
        // a window with more leading ones than the longest code word has bits decodes like the one with
        // exactly that many: rows below 31 - max_len are never needed
        const uint32_t mant = (uint32_t)f.tables.xt_mant;
        d.xt_mant = mant;
        d.xt_row0 = f.max_len < 31u ? 31u - f.max_len : 0u;
        d.xt_low = f.max_len < 32u ? ((1u << (32u - f.max_len)) - 1u) | 1u : 1u;
        d.l1 = reinterpret_cast<const uint2*>(f.dev.xt) + ((size_t)d.xt_row0 << mant);
        d.l1_entries = (32u - d.xt_row0) << mant;
        d.sub_bytes = 0;
        d.tab_kind = 1;
    }
    return d;
}
// Whether a first-level entry can fail to hold the symbol.
static bool table_has_long(const Format& f, const DevFormat& d) {
    return d.tab_kind ? f.tables.xt_unresolved > 0.0 : d.max_len > d.l1_bits;
}
// Share of the symbols whose first-level entry does not hold them.  The kernels that decode three code words
// per window pay a call for every group with such a symbol, so they only take formats where those are rare.
static double table_unresolved_share(const Format& f, const DevFormat& d) {
    return d.tab_kind ? f.tables.xt_unresolved : f.tables.l1_unresolved;
}
constexpr double kGroupedDecodeMaxUnresolved = 1e-4;      // about 2 % of the groups of a warp (2 chains x 3 symbols x 32 lanes)

static void set_pointers(Format& f, void* dev_buf, size_t bytes) {
    const ImageLayout L = image_layout(f);
    unsigned char* b = static_cast<unsigned char*>(dev_buf);
    f.dev.base = dev_buf; f.dev.bytes = bytes;
    f.dev.stream = reinterpret_cast<const uint32_t*>(b + L.stream);
    f.dev.lut = reinterpret_cast<const uint16_t*>(b + L.lut);
    f.dev.l1 = reinterpret_cast<const uint2_host*>(b + L.l1);
    f.dev.sub = reinterpret_cast<const uint2_host*>(b + L.sub);
    f.dev.l1_runs = reinterpret_cast<const uint2_host*>(b + L.l1_runs);
    f.dev.xt = reinterpret_cast<const uint2_host*>(b + L.xt);
    f.dev.rank_value = reinterpret_cast<const float*>(b + L.rank_value);
    f.dev.limit = reinterpret_cast<const uint64_t*>(b + L.limit);
    f.dev.first_left = reinterpret_cast<const uint32_t*>(b + L.first_left);
    f.dev.rank_base = reinterpret_cast<const uint32_t*>(b + L.rank_base);
    f.dev.seg_bit_off = reinterpret_cast<const uint64_t*>(b + L.seg_bit_off);
    f.dev.sub_bits = reinterpret_cast<const uint16_t*>(b + L.sub_bits);
    f.dev.seg_col = reinterpret_cast<const uint32_t*>(b + L.seg_col);
    f.dev.seg_first = reinterpret_cast<const uint32_t*>(b + L.seg_first);
    f.dev.ri = b + L.ri;
    f.dev.cb = reinterpret_cast<const uint32_t*>(b + L.cb);
    f.dev.unit_info = b + L.unit_info;
    f.dev.task_off = reinterpret_cast<const uint64_t*>(b + L.task_off);
    f.dev.task_pos = reinterpret_cast<const uint32_t*>(b + L.task_pos);
}

static int upload(Format& f, void* dev_buf, size_t dev_bytes, void* stream_) {
    if (!dev_buf || (reinterpret_cast<uintptr_t>(dev_buf) & 255u)) return HAC_ERR_INVALID_ARG;
    const ImageLayout L = image_layout(f);
    if (dev_bytes < L.total) return HAC_ERR_BUFFER_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream_);
    unsigned char* b = static_cast<unsigned char*>(dev_buf);
    auto put = [&](size_t off, const void* src, size_t bytes) -> cudaError_t {
        if (bytes == 0) return cudaSuccess;
        return cudaMemcpyAsync(b + off, src, bytes, cudaMemcpyHostToDevice, st);
    };
    HAC_CUDA(cudaMemsetAsync(dev_buf, 0, L.total, st));
    HAC_CUDA(put(L.stream, f.stream.data(), f.stream.size() * 4));
    HAC_CUDA(put(L.lut, f.tables.lut.data(), f.tables.lut.size() * 2));
    HAC_CUDA(put(L.l1, f.tables.l1.data(), f.tables.l1.size() * 4));
    HAC_CUDA(put(L.sub, f.tables.sub.data(), f.tables.sub.size() * 4));
    HAC_CUDA(put(L.l1_runs, f.tables.l1_runs.data(), f.tables.l1_runs.size() * 4));
    HAC_CUDA(put(L.xt, f.tables.xt.data(), f.tables.xt.size() * 4));
    HAC_CUDA(put(L.rank_value, f.tables.rank_value.data(), f.tables.rank_value.size() * 4));
    HAC_CUDA(put(L.limit, f.tables.limit, sizeof(f.tables.limit)));
    HAC_CUDA(put(L.first_left, f.tables.first_left, sizeof(f.tables.first_left)));
    HAC_CUDA(put(L.rank_base, f.tables.rank_base, sizeof(f.tables.rank_base)));
    HAC_CUDA(put(L.seg_bit_off, f.seg_bit_off.data(), f.seg_bit_off.size() * 8));
    HAC_CUDA(put(L.sub_bits, f.sub_bits.data(), f.sub_bits.size() * 2));
    HAC_CUDA(put(L.seg_col, f.seg_col.data(), f.seg_col.size() * 4));
    HAC_CUDA(put(L.seg_first, f.seg_first.data(), f.seg_first.size() * 4));
    if (f.ri_bits == 16) HAC_CUDA(put(L.ri, f.ri16.data(), f.ri16.size() * 2));
    else HAC_CUDA(put(L.ri, f.ri32.data(), f.ri32.size() * 4));
    HAC_CUDA(put(L.cb, f.cb.data(), f.cb.size() * 4));
    HAC_CUDA(put(L.unit_info, f.item_info.data(), f.item_info.size() * 4));
    HAC_CUDA(put(L.task_off, f.task_off.data(), f.task_off.size() * 8));
    HAC_CUDA(put(L.task_pos, f.task_pos.data(), f.task_pos.size() * 4));
    // the source vectors are pageable host memory: wait so they may change or go away afterwards
    HAC_CUDA(cudaStreamSynchronize(st));
    set_pointers(f, dev_buf, dev_bytes);
    return HAC_OK;
}

static int attach(Format& f, void* dev_buf, size_t dev_bytes) {
    if (!dev_buf || (reinterpret_cast<uintptr_t>(dev_buf) & 255u)) return HAC_ERR_INVALID_ARG;
    if (dev_bytes < image_layout(f).total) return HAC_ERR_BUFFER_TOO_SMALL;
    set_pointers(f, dev_buf, dev_bytes);
    return HAC_OK;
}

// Tasks of the tensor-core kernel: runs of consecutive rows of a column (HAC: a sub-segment, S rows; sHAC:
// tc_rows rows, see Format::task_pos).
static uint32_t gemm_task_rows(const Format& f) { return f.sparse ? f.tc_rows : f.S; }
static uint32_t gemm_tasks(const Format& f) {
    const uint32_t t = gemm_task_rows(f);
    return t ? (uint32_t)((f.n + t - 1) / t) : 0u;
}
// Whether a batched sHAC product goes to the tensor-core kernel (zero-filled tiles) rather than to the kernel
// that gathers rows of X: the first costs the dense product, the second nnz * batch * 4 bytes from L2.
static bool shac_tc_wanted(const Format& f, int64_t batch) {
    if (!f.sparse || batch < 2 || f.task_pos.empty() || tune().shac_tc == 0) return false;
    const double tiles = (double)((batch + kGBatch - 1) / kGBatch);
    const double dense_s = (double)f.n * (double)f.m * tiles * kGBatch * 6.0 / 200e12;
    const double gather_s = (double)f.nnz * (double)batch * 4.0 / 5e12;
    return tune().shac_tc == 2 || dense_s < gather_s;
}

// Whether the single-input sHAC kernel can hold the format: it stages two segments' spans and slices of
// ri per warp, which a very large S with 32-bit row indices can push past the shared memory of an SM
// (227 KB on sm_100); such formats take the batched kernel for a single input too.
static bool shac_vec_fits(const Format& f) {
    const size_t per_warp = ((size_t)f.max_unit_chunks * 16 + ((size_t)(32u * f.S * (f.ri_bits / 8) + 15u) / 16u + 1u) * 16u) * 2;
    return 16 + plan_smem_bytes(1u << f.tables.l1_bits, 0, (uint32_t)(f.tables.sub.size() * 4)) + per_warp <= (size_t)232448;
}

// Whether a batched sHAC product may go to the kernel that stages rows of X in shared memory (it needs the row tasks).
static bool shac_rows_possible(const Format& f, int64_t batch) {
    return f.sparse && batch >= 2 && !f.task_pos.empty() && tune().shac_rows != 0;
}

static size_t partial_bytes(const Format& f, int64_t batch) {
    // tensor-core kernel and the kernel that stages rows of X: one partial per row split of the product kernel
    size_t tc = 0;
    if (batch > 1 && (!f.sparse || shac_tc_wanted(f, batch) || shac_rows_possible(f, batch))) {
        const uint32_t t = gemm_tasks(f);
        tc = t > 1 ? (size_t)std::min<uint32_t>(t, kGMaxSplits) * (size_t)f.m * (size_t)batch * 4 : 0;
        if (!f.sparse) return tc;
    }
    // sHAC with one input handles up to two segments of a column in one warp; the batched sHAC kernel
    // and HAC with one input keep one partial per segment
    const bool partials = f.sparse ? f.max_units_per_col > ((batch == 1 && shac_vec_fits(f)) ? 2u : 1u) : f.G > 1;
    return std::max(tc, partials ? f.seg_bit_off.size() * (size_t)batch * 4 : (size_t)0);
}

// Row splits of the tensor-core HAC kernel: 1 (a block owns whole columns and writes y itself)
// unless that leaves most of the SMs idle; a split keeps at least one task per decode chain.
static uint32_t gemm_row_splits(const Format& f, int64_t batch, int sms) {
    const uint64_t blocks = (uint64_t)((f.m + kGCols - 1) / kGCols) * (uint64_t)((batch + kGBatch - 1) / kGBatch);
    const uint32_t tasks = gemm_tasks(f);
    if (blocks * 5 >= (uint64_t)sms * 3 || tasks <= 1) return 1;
    const uint64_t by_sms = std::max<uint64_t>(1, (uint64_t)sms / blocks);
    const uint64_t by_tasks = std::max<uint32_t>(1, tasks / (kGSlots * kGChains));
    return (uint32_t)std::min<uint64_t>(std::min<uint64_t>(by_sms, by_tasks), kGMaxSplits);
}

// Batched HAC: the B tiles of the tensor-core kernel (see hac_pack_x_kernel).  Their number depends on
// the row split, which depends on the device; without a current device (a size query before any CUDA
// call) the split that needs most is assumed.
static uint32_t gemm_max_rounds(const Format& f, uint32_t row_splits) {
    const uint32_t tasks = gemm_tasks(f);
    const uint32_t max_ntl = (tasks + row_splits - 1) / row_splits;
    return (max_ntl + kGChains * kGSlots - 1) / (kGChains * kGSlots);
}
static size_t xpack_bytes(const Format& f, int64_t batch) {
    if (batch <= 1 || f.symbols == 0 || (f.sparse && !shac_tc_wanted(f, batch))) return 0;
    const size_t cpr = (gemm_task_rows(f) + kGChainRows - 1) / kGChainRows;
    size_t tiles = 0;
    DeviceInfo di;
    if (device_info(di) == HAC_OK) {
        const uint32_t rs = gemm_row_splits(f, batch, di.sms);
        tiles = (size_t)rs * kGSlots * gemm_max_rounds(f, rs) * cpr;
    } else {
        for (uint32_t rs = 1; rs <= kGMaxSplits; ++rs)
            tiles = std::max(tiles, (size_t)rs * kGSlots * gemm_max_rounds(f, rs) * cpr);
    }
    return (size_t)((batch + kGBatch - 1) / kGBatch) * tiles * kGXTileBytes;
}

// Batched HAC: start bit of every task of every column, [tasks + 1][m] (see hac_pack_x_kernel).
static size_t task_off_bytes(const Format& f, int64_t batch) {
    if (f.sparse || batch <= 1 || f.symbols == 0 || !f.task_off.empty()) return 0;    // kept in the device image
    return ((size_t)gemm_tasks(f) + 1) * (size_t)f.m * 8;
}

// Workspace of one product: [partial sums, rounded up to 256 bytes][B tiles][task start bits].
static size_t workspace_bytes(const Format& f, int64_t batch) {
    const size_t xp = xpack_bytes(f, batch);
    if (!xp) return partial_bytes(f, batch);
    // never less than a single-input product needs: a batch falls back to those when the tensor-core kernel
    // cannot hold the format's sub-segments
    return std::max(((partial_bytes(f, batch) + 255) & ~(size_t)255) + xp + task_off_bytes(f, batch), partial_bytes(f, 1));
}

// Opt-in to more than 48 KB of dynamic shared memory: once per kernel, device and size.
static int prepare_kernel_ptr(const void* kernel, size_t smem) {
    if (smem <= 48 * 1024) return HAC_OK;
    static std::mutex guard;
    static std::map<std::pair<int, const void*>, size_t> done;
    int dev = 0;
    HAC_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(guard);
    size_t& have = done[std::make_pair(dev, kernel)];
    if (have >= smem) return HAC_OK;
    HAC_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    have = smem;
    return HAC_OK;
}
template <typename K>
static int prepare_kernel(K kernel, size_t smem) { return prepare_kernel_ptr(reinterpret_cast<const void*>(kernel), smem); }

// Resident blocks per SM of a kernel at a block size and shared-memory size: asked once per combination.
static int blocks_per_sm(const void* kernel, int threads, size_t smem, int* out) {
    static std::mutex guard;
    static std::map<std::tuple<int, const void*, int, size_t>, int> known;
    int dev = 0;
    HAC_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(guard);
    auto key = std::make_tuple(dev, kernel, threads, smem);
    auto it = known.find(key);
    if (it == known.end()) {
        int per_sm = 1;
        HAC_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem));
        it = known.emplace(key, std::max(per_sm, 1)).first;
    }
    *out = it->second;
    return HAC_OK;
}

// Launch with programmatic stream serialization: the kernel may start while the one before it in the
// stream drains; it calls depends_wait() before touching anything an earlier kernel may have written.
template <typename... KArgs, typename... Args>
static int launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = tune().pdl != 0 ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 1;
    HAC_CUDA(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
    return HAC_OK;
}

// The same with `cluster_x` consecutive blocks forming a thread-block cluster.
template <typename... KArgs, typename... Args>
static cudaError_t launch_dependent_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                            unsigned cluster_x, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = tune().pdl != 0 ? 1 : 0;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Largest number of warps per block (a multiple of `step`, at most `want`) whose shared memory
// fits; 0 if not even `step` warps fit.
static int fit_warps(size_t fixed, size_t per_warp, int want, int step, size_t budget) {
    for (int w = want; w >= step; w -= step)
        if (fixed + per_warp * (size_t)w <= budget) return w;
    return 0;
}

static int launch_finalize(const Format& f, const DevFormat& d, const float* partial, int64_t batch, float* y,
                           int64_t ys_j, int64_t ys_b, cudaStream_t st, uint32_t direct_up_to) {
    const uint64_t total = (uint64_t)f.m * (uint64_t)batch;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    const int rc = launch_dependent(finalize_kernel, dim3(blocks), dim3(256), 0, st, d, f.sparse, partial, (uint32_t)batch, y,
                                    ys_j, ys_b, direct_up_to);
    if (rc) return rc;
    f.last_launches++;
    return HAC_OK;
}

// Table plan: the widest replication (at most 16 copies) of the level-1 table that fits.
static TablePlan plan_tables(const DevFormat& d, size_t table_budget) {
    TablePlan tp{};
    tp.repl_log2 = 4;
    while (tp.repl_log2 > 0 && plan_smem_bytes(d.l1_entries, tp.repl_log2, d.sub_bytes) > table_budget) tp.repl_log2--;
    return tp;
}

typedef void (*VecKernel)(DevFormat, TablePlan, const float*, int64_t, float*, int64_t, float*);

template <bool kLong>
static VecKernel pick_vec_kernel(const Format& f, int mode, bool x_shared, int chains, bool runs) {
    if (!f.sparse) {
        if (runs) return chains == 2 ? hac_vec_kernel<0, true, kLong, 2, true> : hac_vec_kernel<0, true, kLong, 1, true>;
        if (chains == 2)
            return mode == 1 ? hac_vec_kernel<1, false, kLong, 2, false>
                             : (x_shared ? hac_vec_kernel<0, true, kLong, 2, false>
                                         : hac_vec_kernel<0, false, kLong, 2, false>);
        return mode == 1 ? hac_vec_kernel<1, false, kLong, 1, false>
                         : (x_shared ? hac_vec_kernel<0, true, kLong, 1, false> : hac_vec_kernel<0, false, kLong, 1, false>);
    }
    if (f.ri_bits == 16)
        return mode == 1 ? shac_vec_kernel<1, false, kLong, uint16_t>
                         : (x_shared ? shac_vec_kernel<0, true, kLong, uint16_t>
                                     : shac_vec_kernel<0, false, kLong, uint16_t>);
    return mode == 1 ? shac_vec_kernel<1, false, kLong, uint32_t>
                     : (x_shared ? shac_vec_kernel<0, true, kLong, uint32_t>
                                 : shac_vec_kernel<0, false, kLong, uint32_t>);
}

// ---- single-input HAC with the rows of x in registers -------------------------------------------
constexpr int kRowsS = 64;              // sub-segment length the kernel is compiled for
constexpr int kRowsMaxWarps = 16;

typedef void (*RowsKernel)(DevFormat, TablePlan, const float*, int64_t, float*, int64_t, float*, uint32_t, uint32_t);

template <int kMode, int kTab, int kC>
static RowsKernel pick_rows_kernel3(bool has_long, bool guard) {
    if (has_long) return hac_rows_kernel<kMode, kRowsS, kC, kTab, true, true>;
    return guard ? hac_rows_kernel<kMode, kRowsS, kC, kTab, false, true> : hac_rows_kernel<kMode, kRowsS, kC, kTab, false, false>;
}
template <int kMode, int kTab>
static RowsKernel pick_rows_kernel2(int chains, bool has_long, bool guard) {
    return chains == 3 ? pick_rows_kernel3<kMode, kTab, 3>(has_long, guard) : pick_rows_kernel3<kMode, kTab, 2>(has_long, guard);
}
template <int kMode>
static RowsKernel pick_rows_kernel(bool xt, int chains, bool has_long, bool guard) {
    return xt ? pick_rows_kernel2<kMode, 1>(chains, has_long, guard) : pick_rows_kernel2<kMode, 0>(chains, has_long, guard);
}

struct RowsPlan {
    bool ok = false;
    DevFormat d;
    TablePlan tp;
    unsigned grid = 0;
    int warps = 0, chains = 2;
    size_t smem = 0;
    uint32_t colsum_bytes = 0;
    bool has_long = false;
};

// Whether the rows-in-registers kernel takes this format, and with which block shape: sub-segments of
// kRowsS symbols, no zero-run table in use, enough columns to give every SM some, at least one warp per
// segment position, and tables + two sets of span buffers within an SM's shared memory.  Warps per block
// and chains per lane are the pair that needs the least time by this estimate: the warps of a class share
// the block's columns, `chains` at a time, in rounds; a round costs in proportion to the chains in
// flight on the SM once there are enough of them to fill the instruction issue (about 30), and no less
// than that below.
static RowsPlan plan_rows(const Format& f, const DeviceInfo& di, int mode) {
    RowsPlan pl;
    if (f.sparse || f.S != (uint32_t)kRowsS || f.G == 0 || f.G > (uint32_t)kRowsMaxWarps || tune().rows_kernel == 0) return pl;
    if (mode == 0 && !f.tables.l1_runs.empty() && tune().zero_runs != 0) return pl;
    if ((uint64_t)f.m * 2 < (uint64_t)di.sms) return pl;
    pl.d = dev_format_xt(f);
    pl.has_long = table_has_long(f, pl.d);
    if (table_unresolved_share(f, pl.d) > kGroupedDecodeMaxUnresolved) return pl;
    pl.grid = (unsigned)std::min<int64_t>(di.sms, f.m);
    const uint32_t max_cols = (uint32_t)((f.m + pl.grid - 1) / pl.grid);
    pl.colsum_bytes = (uint32_t)align16((size_t)max_cols * f.G * 4);
    if (pl.colsum_bytes > 16 * 1024) return pl;
    const size_t budget = (size_t)di.max_smem_optin - 256;       // static shared memory of the kernel
    const size_t span = (size_t)f.max_unit_chunks * 16;
    const size_t xs_bytes = mode == 0 ? align16((size_t)f.G * 32 * (kRowsS + 1) * 4) : 0;
    for (int repl = 4; repl >= 0; --repl) {
        const size_t tab = plan_smem_bytes(pl.d.l1_entries, (uint32_t)repl, pl.d.sub_bytes);
        int best_w = 0, best_c = 0;
        uint64_t best_cost = ~0ull;
        for (int chains = 2; chains <= 3; ++chains) {
            // (three chains per lane measured slower than two at the same number of rounds: only on request)
            if (chains != (tune().rows_chains > 0 ? tune().rows_chains : 2)) continue;
            const uint32_t groups = (max_cols + chains - 1) / chains;
            const int max_w = chains == 2 ? kRowsMaxWarps : 12;  // the register budget of the wider kernel
            for (int w = (int)f.G; w <= max_w; ++w) {
                if (tune().rows_warps > 0 && w != tune().rows_warps) continue;
                const size_t set = (size_t)w * chains * span;
                if (tab + pl.colsum_bytes + std::max(2 * set, set + xs_bytes) > budget) break;
                const uint32_t wcls = (uint32_t)w / f.G;             // warps of the least served class
                const uint64_t rounds = (groups + wcls - 1) / wcls;
                // a round is bound by the latency of a lane's serial decode until about 60 chains are in flight
                const uint64_t cost = rounds * (uint64_t)std::max(w * chains, 60);
                if (cost < best_cost || (cost == best_cost && w * chains > best_w * best_c)) {
                    best_cost = cost; best_w = w; best_c = chains;
                }
            }
        }
        // more than two rounds of items per warp: the kernel with x in shared memory, which runs twice the
        // warps, is the faster one
        if (best_w > 0 && best_cost > 2ull * 60 && tune().rows_warps == 0) { if (repl == 4) return pl; continue; }
        if (best_w * best_c >= std::min<int>(16, (int)(f.G * 2)) || (repl == 0 && best_w > 0)) {
            pl.tp = TablePlan{};
            pl.tp.repl_log2 = (uint32_t)repl;
            pl.tp.prefetch = tune().prefetch != 0 ? 1u : 0u;
            pl.warps = best_w;
            pl.chains = best_c;
            const size_t set = (size_t)best_w * best_c * span;
            pl.smem = tab + pl.colsum_bytes + std::max(2 * set, set + xs_bytes);
            pl.ok = true;
            return pl;
        }
    }
    return pl;
}

static int launch_rows(const Format& f, const RowsPlan& pl, int mode, const float* x, int64_t xs_i, float* y,
                       int64_t ys_j, float* aux, cudaStream_t st) {
    const bool guard = 3u * f.max_len > 32u;               // three code words may not fit one window
    RowsKernel kernel = mode == 1 ? pick_rows_kernel<1>(pl.d.tab_kind != 0, pl.chains, pl.has_long, guard)
                                  : pick_rows_kernel<0>(pl.d.tab_kind != 0, pl.chains, pl.has_long, guard);
    int rc = prepare_kernel(kernel, pl.smem);
    if (rc) return rc;
    rc = launch_dependent(kernel, dim3(pl.grid), dim3((unsigned)pl.warps * 32), pl.smem, st, pl.d, pl.tp, x, xs_i, y, ys_j,
                          aux, pl.colsum_bytes, (uint32_t)(f.stream.size() / 4));
    if (rc) return rc;
    HAC_CUDA(cudaGetLastError());
    f.last_launches++;
    return HAC_OK;
}

// ---- single-input sHAC with everything an item needs staged by bulk copies -------------------------
typedef void (*ItemsKernel)(DevFormat, TablePlan, const float*, int64_t, float*, int64_t, float*);

template <int kMode, int kTab, typename RowT>
static ItemsKernel pick_items_kernel3(bool has_long, bool guard) {
    if (kMode == 1 || has_long) return shac_items_kernel<kMode, kTab, true, true, RowT>;     // the test path takes the general one
    return guard ? shac_items_kernel<kMode, kTab, false, true, RowT> : shac_items_kernel<kMode, kTab, false, false, RowT>;
}
template <int kMode, int kTab>
static ItemsKernel pick_items_kernel2(uint32_t ri_bits, bool has_long, bool guard) {
    return ri_bits == 16 ? pick_items_kernel3<kMode, kTab, uint16_t>(has_long, guard)
                         : pick_items_kernel3<kMode, kTab, uint32_t>(has_long, guard);
}
template <int kMode>
static ItemsKernel pick_items_kernel(bool xt, uint32_t ri_bits, bool has_long, bool guard) {
    return xt ? pick_items_kernel2<kMode, 1>(ri_bits, has_long, guard) : pick_items_kernel2<kMode, 0>(ri_bits, has_long, guard);
}

// Launches shac_items_kernel if x, the tables and the staging areas of at least 16 warps fit in an SM's shared
// memory; *launched tells whether it did.
static int launch_items(const Format& f, const DeviceInfo& di, int mode, const float* x, int64_t xs_i, float* y,
                        int64_t ys_j, float* aux, cudaStream_t st, bool* launched) {
    *launched = false;
    if (!f.sparse || tune().items_kernel == 0) return HAC_OK;
    const DevFormat d = dev_format_xt(f);
    if (d.items == 0 || table_unresolved_share(f, d) > kGroupedDecodeMaxUnresolved) return HAC_OK;
    const size_t budget = (size_t)di.max_smem_optin - 256;       // static shared memory of the kernel
    const size_t xbytes = mode == 0 ? align16((size_t)f.n * 4) : 0;
    const size_t ri_stage = mode == 0 ? ((size_t)(32u * f.S * (f.ri_bits / 8) + 15u) / 16u + 1u) * 16u : 0;
    const size_t per_warp = 2 * ((size_t)d.max_unit_chunks * 16 + ri_stage);
    int warps = 0, repl = 4;
    for (; repl >= 0 && !warps; --repl) {
        const size_t tab = plan_smem_bytes(d.l1_entries, (uint32_t)repl, d.sub_bytes);
        for (int w = 32; w >= 16; w -= 4) {
            if (align16(16 + 8 * (size_t)w) + xbytes + tab + per_warp * (size_t)w <= budget) { warps = w; break; }
        }
        if (warps) break;
    }
    if (!warps) return HAC_OK;
    TablePlan tp{};
    tp.repl_log2 = (uint32_t)repl;
    tp.x_bulk = (mode == 0 && xs_i == 1 && (reinterpret_cast<uintptr_t>(x) & 15u) == 0) ? 1u : 0u;
    const size_t smem = align16(16 + 8 * (size_t)warps) + xbytes + plan_smem_bytes(d.l1_entries, tp.repl_log2, d.sub_bytes) +
                        per_warp * (size_t)warps;
    const bool has_long = table_has_long(f, d), guard = 3u * f.max_len > 32u;
    ItemsKernel kernel = mode == 1 ? pick_items_kernel<1>(d.tab_kind != 0, f.ri_bits, has_long, guard)
                                   : pick_items_kernel<0>(d.tab_kind != 0, f.ri_bits, has_long, guard);
    int rc = prepare_kernel(kernel, smem);
    if (rc) return rc;
    const unsigned grid = std::min<unsigned>(d.items, (unsigned)di.sms);
    rc = launch_dependent(kernel, dim3(grid), dim3((unsigned)warps * 32), smem, st, d, tp, x, xs_i, y, ys_j, aux);
    if (rc) return rc;
    HAC_CUDA(cudaGetLastError());
    f.last_launches++;
    *launched = true;
    return HAC_OK;
}

static int launch_vec_shared_x(const Format& f, const DeviceInfo& di, const DevFormat& d_plain, int mode, const float* x,
                               int64_t xs_i, float* y, int64_t ys_j, float* aux, cudaStream_t st, bool* vec_direct,
                               bool allow_group = true);

// mode 0: product with one input; mode 1: debug decode into `aux`.
static int launch_vec(const Format& f, int mode, const float* x, int64_t xs_i, float* y, int64_t ys_j,
                      float* aux, cudaStream_t st, bool* vec_direct = nullptr) {
    DeviceInfo di;
    int rc = device_info(di);
    if (rc) return rc;
    const DevFormat d = dev_format(f);
    if (d.units == 0) return HAC_OK;
    if (!f.sparse) {
        const RowsPlan pl = plan_rows(f, di, mode);
        if (pl.ok) {
            if (vec_direct) *vec_direct = true;
            return launch_rows(f, pl, mode, x, xs_i, y, ys_j, aux, st);
        }
    } else {
        bool launched = false;
        rc = launch_items(f, di, mode, x, xs_i, y, ys_j, aux, st, &launched);
        if (rc || launched) return rc;
    }
    return launch_vec_shared_x(f, di, d, mode, x, xs_i, y, ys_j, aux, st, vec_direct);
}

// The single-input kernels that keep x in shared memory (the general ones).
static int launch_vec_shared_x(const Format& f, const DeviceInfo& di, const DevFormat& d_plain, int mode, const float* x,
                               int64_t xs_i, float* y, int64_t ys_j, float* aux, cudaStream_t st, bool* vec_direct,
                               bool allow_group) {
    int rc = HAC_OK;
    const size_t budget = (size_t)di.max_smem_optin - 256;   // static shared memory of the kernels
    // HAC: two decode chains per lane when two staging areas per warp fit next to a fully
    // replicated table; sHAC: one
    const int chains = f.sparse ? 2 : (d_plain.units > 1 ? 2 : 1);
    // HAC with a first-level table that resolves (nearly) every code word: three code words per window
    bool group = false;
    DevFormat d = d_plain;
    if (allow_group && !f.sparse && mode == 0 && chains == 2 && (f.tables.l1_runs.empty() || tune().zero_runs == 0) &&
        tune().vec_group != 0) {
        const DevFormat dx = dev_format_xt(f);
        if (table_unresolved_share(f, dx) <= kGroupedDecodeMaxUnresolved) { group = true; d = dx; }
    }
    size_t per_warp = (size_t)d.max_unit_chunks * 16 * chains;
    if (f.sparse && mode == 0) per_warp += ((size_t)(32u * f.S * (f.ri_bits / 8) + 15u) / 16u + 1u) * 16u * chains;
    size_t xbytes = 0;
    if (mode == 0) xbytes = f.sparse ? align16((size_t)f.n * 4) : align16(((size_t)f.n + (f.n / f.S + 1)) * 4);
    int want = 32;
    // shared memory: tables + x + per-warp staging.  Prefer keeping x and all warps; give up
    // replicas of the level-1 table before giving up warps (the grouped decoder, whose lookups are most of
    // its shared-memory traffic, gives up to a quarter of the warps first).
    if (group) {
        for (int w = 32; w >= 24; w -= 2)
            if (plan_smem_bytes(d.l1_entries, 4, d.sub_bytes) + xbytes + per_warp * (size_t)w <= budget) { want = w; break; }
    }
    if (tune().vec_warps > 0) want = std::min(32, tune().vec_warps);
    bool x_shared = mode == 0;
    const size_t min_tables = plan_smem_bytes(d.l1_entries, 0, d.sub_bytes) + 16;
    if (x_shared && xbytes + min_tables + per_warp * std::min(want, 8) > budget) { x_shared = false; xbytes = 0; }
    int warps = want;
    while (warps > 1 && xbytes + min_tables + per_warp * (size_t)warps > budget) --warps;
    if (xbytes + min_tables + per_warp * (size_t)warps > budget) return HAC_ERR_BUFFER_TOO_SMALL;
    const size_t fixed = f.sparse ? 16 : 0;                 // mbarrier of the bulk copy of x
    TablePlan tp = plan_tables(d, budget - fixed - xbytes - per_warp * (size_t)warps);
    tp.x_bulk = (f.sparse && mode == 0 && x_shared && xs_i == 1 && (reinterpret_cast<uintptr_t>(x) & 15u) == 0) ? 1u : 0u;
    const size_t smem = fixed + plan_smem_bytes(d.l1_entries, tp.repl_log2, d.sub_bytes) + xbytes + per_warp * warps;
    if (smem > budget) return HAC_ERR_BUFFER_TOO_SMALL;
    const bool has_long = group ? table_has_long(f, d) : d.max_len > d.l1_bits;
    const int threads = warps * 32;
    // HAC with a short code word for zero: the zero-run table replaces the level-1 table
    const bool runs = !f.sparse && mode == 0 && x_shared && !f.tables.l1_runs.empty() && tune().zero_runs != 0;
    DevFormat dk = d;
    if (runs) { dk.l1 = reinterpret_cast<const uint2*>(f.dev.l1_runs); tp.zero_len = f.tables.zero_len; }
    VecKernel kernel = has_long ? pick_vec_kernel<true>(f, mode, x_shared, chains, runs)
                                : pick_vec_kernel<false>(f, mode, x_shared, chains, runs);
    if (group && x_shared && !runs) {
        const bool guard = 3u * f.max_len > 32u;
        if (d.tab_kind)
            kernel = has_long ? hac_vec_kernel<0, true, true, 2, false, true, 1, true>
                              : (guard ? hac_vec_kernel<0, true, false, 2, false, true, 1, true> : hac_vec_kernel<0, true, false, 2, false, true, 1, false>);
        else
            kernel = has_long ? hac_vec_kernel<0, true, true, 2, false, true, 0, true>
                              : (guard ? hac_vec_kernel<0, true, false, 2, false, true, 0, true> : hac_vec_kernel<0, true, false, 2, false, true, 0, false>);
    } else if (group) {
        // x does not fit in shared memory: the plain decoder, which can read it from global memory
        return launch_vec_shared_x(f, di, d_plain, mode, x, xs_i, y, ys_j, aux, st, vec_direct, false);
    }
    rc = prepare_kernel(kernel, smem);
    if (rc) return rc;
    int per_sm = 1;
    rc = blocks_per_sm(reinterpret_cast<const void*>(kernel), threads, smem, &per_sm);
    if (rc) return rc;
    // spread the segments over all SMs (a block's warps take segments blockIdx + k * gridDim)
    const unsigned items = f.sparse ? d.items : (d.units + chains - 1) / chains;
    const unsigned grid = std::min<unsigned>(items, (unsigned)(di.sms * per_sm));
    rc = launch_dependent(kernel, dim3(grid), dim3((unsigned)threads), smem, st, dk, tp, x, xs_i, y, ys_j, aux);
    if (rc) return rc;
    if (vec_direct) *vec_direct = (!f.sparse && (f.G == 1 || (chains == 2 && f.G == 2)));
    HAC_CUDA(cudaGetLastError());
    f.last_launches++;
    return HAC_OK;
}

// Batched HAC product: one block per (128 columns, row split, 64 inputs).
static int launch_gemm_tc(const Format& f, const DeviceInfo& di, const DevFormat&, const float* x, int64_t xs_i,
                          int64_t xs_b, int64_t batch, float* y, int64_t ys_j, int64_t ys_b, float* partial,
                          unsigned char* xpack, cudaStream_t st, uint32_t* row_splits_out) {
    DevFormat d = dev_format_xt(f);
    const bool has_long = table_has_long(f, d);
    const int sp = f.sparse ? (int)(f.ri_bits / 8) : 0;
    if (f.sparse) d.S = f.tc_rows;               // the kernels' task length
    auto pick = [&](auto tab, auto lng) {
        constexpr int kTab = decltype(tab)::value;
        constexpr bool kLng = decltype(lng)::value;
        return sp == 0 ? hac_gemm_tc_kernel<kTab, kLng, 0> : (sp == 2 ? hac_gemm_tc_kernel<kTab, kLng, 2> : hac_gemm_tc_kernel<kTab, kLng, 4>);
    };
    auto kernel = d.tab_kind ? (has_long ? pick(std::integral_constant<int, 1>(), std::true_type()) : pick(std::integral_constant<int, 1>(), std::false_type()))
                             : (has_long ? pick(std::integral_constant<int, 0>(), std::true_type()) : pick(std::integral_constant<int, 0>(), std::false_type()));
    const size_t budget = (size_t)di.max_smem_optin;
    const uint32_t slot_bytes = (f.sparse ? f.max_task_chunks : d.max_sub_chunks) * 16;
    const uint32_t rslot_bytes = f.sparse ? f.max_task_ri_chunks * 16 : 0;
    // shared memory: double stream buffers if they still leave room for a level-1 table with 8 replicas,
    // else single ones with the widest table that fits
    uint32_t nbuf = 0;
    size_t fixed = 0;
    for (uint32_t want_repl : {3u, 2u, 1u, 0u}) {
        for (uint32_t nb : {2u, 1u}) {
            // the stream buffers double as the epilogue's four 32 x 33 transpose tiles
            // the stream buffers double as the epilogue's tiles (four 32 x 33 transposes, or the 128 x 65 sums)
            const size_t fx = 256 + 128 + (size_t)kGSlots * kGStages * kGXTileBytes +
                              std::max<size_t>((size_t)kGDecodeWarps * nb * kGChains * 32 * (slot_bytes + rslot_bytes),
                                               (size_t)kGCols * (kGBatch + 1) * 4);
            if (fx + plan_smem_bytes(d.l1_entries, want_repl, d.sub_bytes) <= budget) { nbuf = nb; fixed = fx; break; }
        }
        if (nbuf) break;
    }
    if (!nbuf) return HAC_ERR_BUFFER_TOO_SMALL;
    const TablePlan tp = plan_tables(d, budget - fixed);
    // the block allocates all of tensor memory: ask for enough shared memory that no second block shares the SM
    const size_t smem = std::max(fixed + plan_smem_bytes(d.l1_entries, tp.repl_log2, d.sub_bytes), budget / 2 + 1024);
    int rc = prepare_kernel(kernel, smem);
    if (rc) return rc;
    const uint32_t col_blocks = (uint32_t)((f.m + kGCols - 1) / kGCols);
    const uint32_t batch_tiles = (uint32_t)((batch + kGBatch - 1) / kGBatch);
    const uint32_t rs = gemm_row_splits(f, batch, di.sms);
    const uint64_t grid = (uint64_t)col_blocks * rs * batch_tiles;
    if (grid > 0x7fffffffull) return HAC_ERR_OFFSET_OVERFLOW;
    const uint32_t tasks = gemm_tasks(f), cpr = (d.S + kGChainRows - 1) / kGChainRows;
    const uint32_t max_rounds = gemm_max_rounds(f, rs);
    const uint64_t pack_blocks = (uint64_t)batch_tiles * rs * kGSlots * max_rounds * cpr;
    if (pack_blocks > 0x7fffffffull) return HAC_ERR_OFFSET_OVERFLOW;
    // the B tiles are a multiple of 8 bytes, so the start bits that follow them are aligned
    if (f.sparse && f.task_off.empty()) return HAC_ERR_BUFFER_TOO_SMALL;
    const bool cached_off = !f.task_off.empty();
    uint64_t* task_off = cached_off ? const_cast<uint64_t*>(f.dev.task_off)
                                    : reinterpret_cast<uint64_t*>(xpack + xpack_bytes(f, batch));
    const uint64_t off_blocks = cached_off ? 0 : ((uint64_t)d.G * d.m + 255) / 256;
    if (pack_blocks + off_blocks > 0x7fffffffull) return HAC_ERR_OFFSET_OVERFLOW;
    rc = launch_dependent(hac_pack_x_kernel, dim3((unsigned)(pack_blocks + off_blocks)), dim3(256), 0, st, d, x, xs_i, xs_b,
                          (uint32_t)batch, xpack, tasks, rs, max_rounds, cpr, (uint32_t)pack_blocks, task_off);
    if (rc) return rc;
    f.last_launches++;
    // The row splits of a column block form a thread-block cluster that adds its sums through distributed
    // shared memory; if the device refuses the cluster, they go to the workspace and a finishing kernel adds them.
    bool clustered = false;
    if (rs > 1 && tune().gemm_cluster != 0) {
        const cudaError_t ce = launch_dependent_cluster(kernel, dim3((unsigned)grid), dim3(kGWarps * 32), smem, st, rs, d, tp,
                                                        (const unsigned char*)xpack, (uint32_t)batch, y, ys_j, ys_b, partial,
                                                        (const uint64_t*)task_off, col_blocks, rs, max_rounds, slot_bytes, nbuf, 1u,
                                                        f.dev.task_pos, rslot_bytes);
        if (ce == cudaSuccess) clustered = true;
        else (void)cudaGetLastError();
    }
    if (!clustered) {
        rc = launch_dependent(kernel, dim3((unsigned)grid), dim3(kGWarps * 32), smem, st, d, tp,
                              (const unsigned char*)xpack, (uint32_t)batch, y, ys_j, ys_b, partial, (const uint64_t*)task_off,
                              col_blocks, rs, max_rounds, slot_bytes, nbuf, 0u, f.dev.task_pos, rslot_bytes);
        if (rc) return rc;
    }
    f.last_launches++;
    *row_splits_out = clustered ? 1u : rs;       // 1: the outputs are written, nothing to finish
    return HAC_OK;
}

template <int kAcc>
static int launch_batch_t(const Format& f, const DeviceInfo& di, const DevFormat& d, const float* x, int64_t xs_i,
                          int64_t xs_b, int64_t batch, float* y, int64_t ys_j, int64_t ys_b, float* partial,
                          cudaStream_t st) {
    const size_t budget = (size_t)di.max_smem_optin;
    const TablePlan tp = plan_tables(d, std::max<size_t>(32 * 1024, plan_smem_bytes(d.l1_entries, 0, d.sub_bytes)));
    const size_t tab = plan_smem_bytes(d.l1_entries, tp.repl_log2, d.sub_bytes);
    constexpr uint32_t kTile = 32 * kAcc;
    const uint32_t batch_tiles = (uint32_t)((batch + kTile - 1) / kTile);
    const size_t per_warp = (size_t)d.max_unit_chunks * 16 + 2 * kBatchRows * 4;
    const int warps = fit_warps(tab + 32, per_warp, 8, 1, budget);
    if (warps == 0) return HAC_ERR_BUFFER_TOO_SMALL;
    const size_t smem = tab + 32 + per_warp * warps;
    void (*kernel)(DevFormat, TablePlan, const float*, int64_t, int64_t, uint32_t, float*, int64_t, int64_t,
                   float*, uint32_t) = f.ri_bits == 16 ? shac_batch_kernel<kAcc, uint16_t> : shac_batch_kernel<kAcc, uint32_t>;
    int rc = prepare_kernel(kernel, smem);
    if (rc) return rc;
    int per_sm = 1;
    rc = blocks_per_sm(reinterpret_cast<const void*>(kernel), warps * 32, smem, &per_sm);
    if (rc) return rc;
    const uint64_t items = (uint64_t)d.units * batch_tiles;
    const unsigned grid = (unsigned)std::min<uint64_t>((items + warps - 1) / warps, (uint64_t)di.sms * per_sm);
    // up to 16 inputs: the smallest power of two that holds them, as lanes per entry
    uint32_t narrow = 0;
    if (batch <= 16) { narrow = 2; while ((int64_t)narrow < batch) narrow <<= 1; }
    kernel<<<grid, warps * 32, smem, st>>>(d, tp, x, xs_i, xs_b, (uint32_t)batch, y, ys_j, ys_b, partial, narrow);
    HAC_CUDA(cudaGetLastError());
    f.last_launches++;
    return HAC_OK;
}

// Batched sHAC through shac_rowblock_kernel.  Returns HAC_ERR_BUFFER_TOO_SMALL (nothing launched) when the format,
// the layout of X or the estimate says that another kernel should take the product.  *splits_out: row splits whose
// sums rowblock_finalize_kernel has added (0: y was written directly).
static int launch_shac_rows(const Format& f, const DeviceInfo& di, const DevFormat& d0, const float* x, int64_t xs_i,
                            int64_t xs_b, int64_t batch, float* y, int64_t ys_j, int64_t ys_b, float* partial,
                            cudaStream_t st) {
    if (!shac_rows_possible(f, batch) || xs_b != 1 || batch > ((int64_t)1 << 22)) return HAC_ERR_BUFFER_TOO_SMALL;
    DevFormat d = d0;
    d.S = f.tc_rows;
    const int in = batch > 64 ? 4 : (batch > 32 ? 2 : 1);
    const uint32_t tile_b = 32u * (uint32_t)in;
    const uint32_t tiles = (uint32_t)((batch + tile_b - 1) / tile_b);
    const size_t budget = (size_t)di.max_smem_optin;
    TablePlan tp = plan_tables(d, 32 * 1024);
    const size_t tab = plan_smem_bytes(d.l1_entries, tp.repl_log2, d.sub_bytes) + 16 + kRbListBytes;
    const uint32_t tasks = gemm_tasks(f);
    // tasks per group: as many rows of X as shared memory holds (a multiple of the four tasks of a pass where possible),
    // in one buffer; two buffers of half that when a group is still at least a pass
    const size_t task_bytes = (size_t)d.S * tile_b * 4;
    if (tab + task_bytes > budget) return HAC_ERR_BUFFER_TOO_SMALL;
    uint32_t group = (uint32_t)std::min<size_t>((budget - tab) / task_bytes, tasks), nbuf = 1;
    const uint32_t wc = 8u, pass = 32u / wc;      // columns per warp, tasks per pass
    if (group >= 2 * pass) { group = (group / 2) / pass * pass; nbuf = 2; }
    else if (group >= pass) group = group / pass * pass;
    if (tune().shac_rows_group > 0 && (size_t)tune().shac_rows_group * task_bytes + tab <= budget) {
        group = (uint32_t)tune().shac_rows_group;
        nbuf = 2 * (size_t)group * task_bytes + tab <= budget ? 2u : 1u;
    }
    const size_t xbytes = (size_t)group * task_bytes;
    const uint32_t col_blocks = (uint32_t)((f.m + kRbWarps * wc - 1) / (kRbWarps * wc));
    const uint64_t blocks = (uint64_t)col_blocks * tiles;
    uint32_t rs = 1;
    if (blocks * 5 < (uint64_t)di.sms * 3 && tasks > 1)
        rs = (uint32_t)std::min<uint64_t>(std::min<uint64_t>(std::max<uint64_t>(1, (uint64_t)di.sms / blocks), tasks), kGMaxSplits);      // one wave
    // Measured on a 25088 x 4096 layer with 96 % zeros: 99 / 157 / 282 us for 32 / 64 / 128 inputs against 127 / 219 / 390 us
    // for the other two kernels, but slower than they are for 16 inputs (102 against 77 us) and for moderately sparse layers
    // (whose row tasks are short), so: a tile's worth of inputs and at most one weight in eight stored.
    if (tune().shac_rows != 2 && (batch < 28 || (double)f.nnz * 8.0 > (double)f.n * (double)f.m)) return HAC_ERR_BUFFER_TOO_SMALL;
    const uint32_t aligned = (reinterpret_cast<uintptr_t>(x) % 16 == 0 && xs_i % 4 == 0) ? 1u : 0u;
    typedef void (*RowsKernel)(DevFormat, TablePlan, const float*, int64_t, uint32_t, float*, int64_t, int64_t, float*,
                               const uint64_t*, const uint32_t*, uint32_t, uint32_t, uint32_t, uint32_t, uint32_t, uint32_t);
    RowsKernel kernel;
    if (f.ri_bits == 16)
        kernel = in == 4 ? shac_rowblock_kernel<4, 8, uint16_t> : (in == 2 ? shac_rowblock_kernel<2, 8, uint16_t> : shac_rowblock_kernel<1, 8, uint16_t>);
    else
        kernel = in == 4 ? shac_rowblock_kernel<4, 8, uint32_t> : (in == 2 ? shac_rowblock_kernel<2, 8, uint32_t> : shac_rowblock_kernel<1, 8, uint32_t>);
    const size_t smem = tab + nbuf * xbytes;
    int rc = prepare_kernel(kernel, smem);
    if (rc) return rc;
    rc = launch_dependent(kernel, dim3(col_blocks * rs, tiles), dim3(kRbWarps * 32), smem, st, d, tp, x, xs_i, (uint32_t)batch, y,
                          ys_j, ys_b, partial, f.dev.task_off, f.dev.task_pos, tasks, rs, col_blocks, nbuf, aligned, group);
    if (rc) return rc;
    f.last_launches++;
    if (rs > 1) {
        const uint64_t total = (uint64_t)f.m * (uint64_t)batch;
        const unsigned grid = (unsigned)std::min<uint64_t>((total + 255) / 256, (uint64_t)di.sms * 8);
        rc = launch_dependent(rowblock_finalize_kernel, dim3(grid), dim3(256), 0, st, (const float*)partial, rs, (uint32_t)f.m,
                              (uint32_t)batch, y, ys_j, ys_b, f.epi_bias, (uint32_t)f.epi_relu);
        if (rc) return rc;
        f.last_launches++;
    }
    return HAC_OK;
}

static int dot(const Format& f, const float* x, int64_t batch, int64_t xs_i, int64_t xs_b, float* y,
               int64_t ys_j, int64_t ys_b, void* workspace, size_t workspace_bytes_given, void* stream_,
               const hac_epilogue* epi = nullptr) {
    if (!f.dev.base) return HAC_ERR_NOT_UPLOADED;
    if (epi && epi->reserved != 0) return HAC_ERR_INVALID_ARG;
    // the epilogue rides in the kernel-side view of the format for the duration of this call
    struct EpilogueScope {
        const Format& f;
        EpilogueScope(const Format& f_, const hac_epilogue* e) : f(f_) { f.epi_bias = e ? e->bias : nullptr; f.epi_relu = e ? (e->relu != 0) : 0; }
        ~EpilogueScope() { f.epi_bias = nullptr; f.epi_relu = 0; }
    } scope(f, epi);
    if (!x || !y || batch < 1 || batch > ((int64_t)1 << 24)) return HAC_ERR_INVALID_ARG;
    const size_t need = workspace_bytes(f, batch);
    if (need > 0 && (!workspace || workspace_bytes_given < need)) return HAC_ERR_BUFFER_TOO_SMALL;
    if (need > 0 && (reinterpret_cast<uintptr_t>(workspace) & 15u)) return HAC_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream_);
    f.last_launches = 0;
    float* partial = static_cast<float*>(workspace);
    const DevFormat d = dev_format(f);
    int rc = HAC_OK;
    bool direct = false;                     // the product kernel wrote every output itself
    uint32_t gemm_splits = 0;                // batched HAC: row splits used (1 = outputs written directly)
    bool wide_single = false;                // sHAC, one input, through the batched kernel (see shac_vec_fits)
    bool shac_tc = false;                    // sHAC batch through the tensor-core kernel
    bool shac_rows = false;                  // sHAC batch through the kernel that stages rows of X (it finishes y itself)
    if (d.units > 0) {
        if (batch == 1 && (!f.sparse || shac_vec_fits(f))) {
            rc = launch_vec(f, 0, x, xs_i, y, ys_j, partial, st, &direct);
        } else if (batch == 1) {
            DeviceInfo di;
            rc = device_info(di);
            if (rc) return rc;
            rc = launch_batch_t<1>(f, di, d, x, xs_i, xs_b, batch, y, ys_j, ys_b, partial, st);
            wide_single = true;
        } else {
            DeviceInfo di;
            rc = device_info(di);
            if (rc) return rc;
            if (!f.sparse) {
                unsigned char* xpack = static_cast<unsigned char*>(workspace) + ((partial_bytes(f, batch) + 255) & ~(size_t)255);
                rc = launch_gemm_tc(f, di, d, x, xs_i, xs_b, batch, y, ys_j, ys_b, partial, xpack, st, &gemm_splits);
                if (rc == HAC_ERR_BUFFER_TOO_SMALL) {
                    // Sub-segments too long for the per-lane stream buffers of the tensor-core kernel (a very
                    // large S): one single-input product per input instead.  Slow, but every format works.
                    rc = HAC_OK;
                    for (int64_t b = 0; b < batch && rc == HAC_OK; ++b) {
                        bool wrote_y = false;
                        rc = launch_vec(f, 0, x + b * xs_b, xs_i, y + b * ys_b, ys_j, partial, st, &wrote_y);
                        if (rc == HAC_OK && f.G > 1 && !wrote_y)
                            rc = launch_finalize(f, d, partial, 1, y + b * ys_b, ys_j, 0, st, 1);
                    }
                }
            } else if ((rc = launch_shac_rows(f, di, d, x, xs_i, xs_b, batch, y, ys_j, ys_b, partial, st)) != HAC_ERR_BUFFER_TOO_SMALL) {
                shac_rows = true;                    // launched (or failed for good)
            } else if ((rc = HAC_OK, shac_tc_wanted(f, batch)) && [&]() {
                           // moderately sparse, or a large batch: the tensor-core kernel with zero-filled tiles
                           unsigned char* xpack = static_cast<unsigned char*>(workspace) + ((partial_bytes(f, batch) + 255) & ~(size_t)255);
                           rc = launch_gemm_tc(f, di, d, x, xs_i, xs_b, batch, y, ys_j, ys_b, partial, xpack, st, &gemm_splits);
                           if (rc == HAC_ERR_BUFFER_TOO_SMALL) { rc = HAC_OK; gemm_splits = 0; return false; }
                           shac_tc = true;
                           return true;
                       }()) {
            } else {
                const int acc = (int)std::min<int64_t>(kAccMax, (batch + 31) / 32);
                switch (acc) {
                    case 1: rc = launch_batch_t<1>(f, di, d, x, xs_i, xs_b, batch, y, ys_j, ys_b, partial, st); break;
                    case 2: rc = launch_batch_t<2>(f, di, d, x, xs_i, xs_b, batch, y, ys_j, ys_b, partial, st); break;
                    case 3: rc = launch_batch_t<3>(f, di, d, x, xs_i, xs_b, batch, y, ys_j, ys_b, partial, st); break;
                    default: rc = launch_batch_t<4>(f, di, d, x, xs_i, xs_b, batch, y, ys_j, ys_b, partial, st); break;
                }
            }
        }
        if (rc) return rc;
    }
    // columns the product kernel did not finish itself (several segments, or none at all)
    uint32_t direct_up_to = 1;
    bool finish;
    DevFormat dfin = d;
    if (shac_rows) {
        finish = false;
    } else if ((!f.sparse && batch > 1) || shac_tc) {
        if (gemm_splits > 1) {               // partial[split][b][j]
            dim3 grid((unsigned)((f.m + 31) / 32), (unsigned)((batch + 31) / 32));
            // launched the ordinary way: started early, its blocks only took the idle SMs from the product
            // kernel's successor (measured: slower)
            gemm_finalize_kernel<<<grid, dim3(32, 8), 0, st>>>(partial, gemm_splits, (uint32_t)f.m, (uint32_t)batch, y,
                                                               ys_j, ys_b, f.epi_bias, f.epi_relu);
            HAC_CUDA(cudaGetLastError());
            f.last_launches++;
        }
        finish = false;
    } else if (!f.sparse) {
        finish = f.G > 1 && !direct;
    } else if (batch == 1 && !wide_single) {
        direct_up_to = 2;
        finish = f.max_units_per_col > 2 || f.has_empty_col;
    } else {
        finish = f.max_units_per_col > 1 || f.has_empty_col;
    }
    if (finish || d.units == 0) rc = launch_finalize(f, dfin, partial, batch, y, ys_j, ys_b, st, direct_up_to);
    return rc;
}

static size_t host_scratch_bytes(const Format& f, int64_t batch) {
    const size_t xb = align16((size_t)batch * f.n * 4 + 240) ;
    const size_t yb = align16((size_t)batch * f.m * 4 + 240);
    const size_t extra = (batch > 1 && f.sparse) ? xb : 0;  // sHAC: transposed copy of X (its batched kernel gathers rows of X)
    return xb + extra + yb + align16(workspace_bytes(f, batch)) + 1024;
}

static int dot_host(const Format& f, const float* X, int64_t batch, float* Y, void* scratch, size_t scratch_bytes,
                    void* stream_, bool wait) {
    if (!f.dev.base) return HAC_ERR_NOT_UPLOADED;
    if (!X || !Y || !scratch || batch < 1) return HAC_ERR_INVALID_ARG;
    if (scratch_bytes < host_scratch_bytes(f, batch)) return HAC_ERR_BUFFER_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream_);
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    unsigned char* b = static_cast<unsigned char*>(scratch);
    b = reinterpret_cast<unsigned char*>(up(reinterpret_cast<uintptr_t>(b)));
    float* xd = reinterpret_cast<float*>(b);
    b += up((size_t)batch * f.n * 4);
    float* xt = xd;
    const bool transpose = batch > 1 && f.sparse;
    if (transpose) { xt = reinterpret_cast<float*>(b); b += up((size_t)batch * f.n * 4); }
    float* yd = reinterpret_cast<float*>(b);
    b += up((size_t)batch * f.m * 4);
    void* ws = b;
    HAC_CUDA(cudaMemcpyAsync(xd, X, (size_t)batch * f.n * 4, cudaMemcpyHostToDevice, st));
    int extra = 0;
    int rc;
    if (transpose) {
        dim3 grid((unsigned)((f.n + 31) / 32), (unsigned)((batch + 31) / 32));
        transpose_kernel<<<grid, dim3(32, 8), 0, st>>>(xd, xt, (uint32_t)batch, (uint32_t)f.n);
        HAC_CUDA(cudaGetLastError());
        extra = 1;
        rc = dot(f, xt, batch, batch, 1, yd, 1, f.m, ws, workspace_bytes(f, batch), stream_);
    } else {
        // X is used as it lies, one input per row: the kernels take element strides
        rc = dot(f, xd, batch, 1, f.n, yd, 1, f.m, ws, workspace_bytes(f, batch), stream_);
    }
    if (rc) return rc;
    f.last_launches += extra;
    HAC_CUDA(cudaMemcpyAsync(Y, yd, (size_t)batch * f.m * 4, cudaMemcpyDeviceToHost, st));
    if (wait) HAC_CUDA(cudaStreamSynchronize(st));
    return HAC_OK;
}

// Scratch of hac_dot_noalloc: part of the library image, one copy per device that loads it.
static __device__ __align__(256) unsigned char g_noalloc_scratch[HAC_NOALLOC_SCRATCH_BYTES];

// Device address of g_noalloc_scratch on the current device, looked up once per device.  In host
// code the array's name only stands for the symbol; the kernels need the address this returns.
static int noalloc_scratch_address(void** out) {
    static std::mutex guard;
    static void* address[64] = {};
    int dev = 0;
    HAC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return HAC_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(guard);
    if (!address[dev]) {
        void* ptr = nullptr;
        HAC_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
        if (!ptr) return HAC_ERR_CUDA;
        address[dev] = ptr;
    }
    *out = address[dev];
    return HAC_OK;
}

static int dot_noalloc(const Format& f, const float* x, int64_t batch, int64_t xs_i, int64_t xs_b, float* y,
                       int64_t ys_j, int64_t ys_b, void* stream_) {
    if (!f.dev.base) return HAC_ERR_NOT_UPLOADED;
    if (!x || !y || batch < 1 || batch > ((int64_t)1 << 24)) return HAC_ERR_INVALID_ARG;
    const size_t need = workspace_bytes(f, batch);
    if (need > (size_t)HAC_NOALLOC_SCRATCH_BYTES) {
        g_last_cuda_error = "hac_dot_noalloc: this product needs " + std::to_string(need) +
                            " bytes of workspace, the built-in buffer holds " +
                            std::to_string((size_t)HAC_NOALLOC_SCRATCH_BYTES);
        return HAC_ERR_BUFFER_TOO_SMALL;
    }
    void* scratch = nullptr;
    const int rc = noalloc_scratch_address(&scratch);
    if (rc != HAC_OK) return rc;
    return dot(f, x, batch, xs_i, xs_b, y, ys_j, ys_b, scratch, (size_t)HAC_NOALLOC_SCRATCH_BYTES, stream_);
}

static int debug_decode(const Format& f, float* out, void* stream_) {
    if (!f.dev.base) return HAC_ERR_NOT_UPLOADED;
    if (!out) return HAC_ERR_INVALID_ARG;
    f.last_launches = 0;
    return launch_vec(f, 1, nullptr, 0, nullptr, 0, out, static_cast<cudaStream_t>(stream_));
}

}  // namespace hacb200

using namespace hacb200;

extern "C" {

int hac_device_bytes(const hac_format* f, size_t* out) {
    if (!f || !out) return HAC_ERR_INVALID_ARG;
    *out = image_layout(f->f).total;
    return HAC_OK;
}
int shac_device_bytes(const shac_format* f, size_t* out) {
    if (!f || !out) return HAC_ERR_INVALID_ARG;
    *out = image_layout(f->f).total;
    return HAC_OK;
}
int hac_upload(hac_format* f, void* dev_buf, size_t dev_bytes, void* cuda_stream) {
    return f ? upload(f->f, dev_buf, dev_bytes, cuda_stream) : HAC_ERR_INVALID_ARG;
}
int shac_upload(shac_format* f, void* dev_buf, size_t dev_bytes, void* cuda_stream) {
    return f ? upload(f->f, dev_buf, dev_bytes, cuda_stream) : HAC_ERR_INVALID_ARG;
}
int hac_attach(hac_format* f, void* dev_buf, size_t dev_bytes) {
    return f ? attach(f->f, dev_buf, dev_bytes) : HAC_ERR_INVALID_ARG;
}
int shac_attach(shac_format* f, void* dev_buf, size_t dev_bytes) {
    return f ? attach(f->f, dev_buf, dev_bytes) : HAC_ERR_INVALID_ARG;
}

int hac_workspace_bytes(const hac_format* f, int64_t batch, size_t* out) {
    if (!f || !out || batch < 1) return HAC_ERR_INVALID_ARG;
    *out = workspace_bytes(f->f, batch);
    return HAC_OK;
}
int shac_workspace_bytes(const shac_format* f, int64_t batch, size_t* out) {
    if (!f || !out || batch < 1) return HAC_ERR_INVALID_ARG;
    *out = workspace_bytes(f->f, batch);
    return HAC_OK;
}

int hac_dot(const hac_format* f, const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b, float* y,
            int64_t y_stride_j, int64_t y_stride_b, void* workspace, size_t workspace_bytes_, void* cuda_stream) {
    if (!f) return HAC_ERR_INVALID_ARG;
    return dot(f->f, x, batch, x_stride_i, x_stride_b, y, y_stride_j, y_stride_b, workspace, workspace_bytes_,
               cuda_stream);
}
int shac_dot(const shac_format* f, const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b, float* y,
             int64_t y_stride_j, int64_t y_stride_b, void* workspace, size_t workspace_bytes_, void* cuda_stream) {
    if (!f) return HAC_ERR_INVALID_ARG;
    return dot(f->f, x, batch, x_stride_i, x_stride_b, y, y_stride_j, y_stride_b, workspace, workspace_bytes_,
               cuda_stream);
}

int hac_dot_layer(const hac_format* f, const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b, float* y,
                  int64_t y_stride_j, int64_t y_stride_b, const hac_epilogue* epilogue, void* workspace,
                  size_t workspace_bytes_, void* cuda_stream) {
    if (!f) return HAC_ERR_INVALID_ARG;
    return dot(f->f, x, batch, x_stride_i, x_stride_b, y, y_stride_j, y_stride_b, workspace, workspace_bytes_,
               cuda_stream, epilogue);
}
int shac_dot_layer(const shac_format* f, const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b, float* y,
                   int64_t y_stride_j, int64_t y_stride_b, const hac_epilogue* epilogue, void* workspace,
                   size_t workspace_bytes_, void* cuda_stream) {
    if (!f) return HAC_ERR_INVALID_ARG;
    return dot(f->f, x, batch, x_stride_i, x_stride_b, y, y_stride_j, y_stride_b, workspace, workspace_bytes_,
               cuda_stream, epilogue);
}

// A stack of layers as one chained submission: layer l reads the activations layer l - 1 wrote.
int hac_chain(const hac_layer* layers, int n_layers, const float* x, int64_t batch, float* y, float* act0, float* act1,
              size_t act_floats, void* workspace, size_t workspace_bytes_, void* cuda_stream) {
    if (!layers || n_layers < 1 || !x || !y || batch < 1) return HAC_ERR_INVALID_ARG;
    // shapes must chain, and the two activation buffers must hold the widest intermediate result
    for (int l = 0; l < n_layers; ++l) {
        if ((layers[l].hac != nullptr) == (layers[l].shac != nullptr)) return HAC_ERR_INVALID_ARG;
        const Format& f = layers[l].hac ? layers[l].hac->f : layers[l].shac->f;
        if (l > 0) {
            const Format& p = layers[l - 1].hac ? layers[l - 1].hac->f : layers[l - 1].shac->f;
            if (p.m != f.n) return HAC_ERR_INVALID_ARG;
        }
        if (l + 1 < n_layers) {
            if (!act0 || (n_layers > 2 && !act1)) return HAC_ERR_INVALID_ARG;
            if ((size_t)f.m * (size_t)batch > act_floats) return HAC_ERR_BUFFER_TOO_SMALL;
        }
        if (workspace_bytes(f, batch) > workspace_bytes_) return HAC_ERR_BUFFER_TOO_SMALL;
    }
    const float* in = x;
    int launches = 0;
    for (int l = 0; l < n_layers; ++l) {
        const Format& f = layers[l].hac ? layers[l].hac->f : layers[l].shac->f;
        float* out = l + 1 == n_layers ? y : ((l & 1) ? act1 : act0);
        // activations are [features][batch], inputs of a batch contiguous (a plain vector for one input)
        const int rc = dot(f, in, batch, batch, 1, out, batch, 1, workspace, workspace_bytes_, cuda_stream, &layers[l].epilogue);
        if (rc) return rc;
        launches += f.last_launches;
        in = out;
    }
    const Format& last = layers[n_layers - 1].hac ? layers[n_layers - 1].hac->f : layers[n_layers - 1].shac->f;
    last.last_launches = launches;               // the whole chain, reported through the last layer's handle
    return HAC_OK;
}

int hac_dot_noalloc(const hac_format* f, const float* x, int64_t batch, int64_t x_stride_i, int64_t x_stride_b,
                    float* y, int64_t y_stride_j, int64_t y_stride_b, void* cuda_stream) {
    if (!f) return HAC_ERR_INVALID_ARG;
    return dot_noalloc(f->f, x, batch, x_stride_i, x_stride_b, y, y_stride_j, y_stride_b, cuda_stream);
}

int hac_dot_host_scratch_bytes(const hac_format* f, int64_t batch, size_t* out) {
    if (!f || !out || batch < 1) return HAC_ERR_INVALID_ARG;
    *out = host_scratch_bytes(f->f, batch);
    return HAC_OK;
}
int shac_dot_host_scratch_bytes(const shac_format* f, int64_t batch, size_t* out) {
    if (!f || !out || batch < 1) return HAC_ERR_INVALID_ARG;
    *out = host_scratch_bytes(f->f, batch);
    return HAC_OK;
}
int hac_dot_host(const hac_format* f, const float* X_host, int64_t batch, float* Y_host, void* dev_scratch,
                 size_t dev_scratch_bytes, void* cuda_stream) {
    if (!f) return HAC_ERR_INVALID_ARG;
    return dot_host(f->f, X_host, batch, Y_host, dev_scratch, dev_scratch_bytes, cuda_stream, true);
}
int shac_dot_host(const shac_format* f, const float* X_host, int64_t batch, float* Y_host, void* dev_scratch,
                  size_t dev_scratch_bytes, void* cuda_stream) {
    if (!f) return HAC_ERR_INVALID_ARG;
    return dot_host(f->f, X_host, batch, Y_host, dev_scratch, dev_scratch_bytes, cuda_stream, true);
}
int hac_dot_host_async(const hac_format* f, const float* X_host, int64_t batch, float* Y_host, void* dev_scratch,
                       size_t dev_scratch_bytes, void* cuda_stream) {
    if (!f) return HAC_ERR_INVALID_ARG;
    return dot_host(f->f, X_host, batch, Y_host, dev_scratch, dev_scratch_bytes, cuda_stream, false);
}
int shac_dot_host_async(const shac_format* f, const float* X_host, int64_t batch, float* Y_host, void* dev_scratch,
                        size_t dev_scratch_bytes, void* cuda_stream) {
    if (!f) return HAC_ERR_INVALID_ARG;
    return dot_host(f->f, X_host, batch, Y_host, dev_scratch, dev_scratch_bytes, cuda_stream, false);
}

int hac_debug_decode(const hac_format* f, float* W_colmajor_dev, void* cuda_stream) {
    return f ? debug_decode(f->f, W_colmajor_dev, cuda_stream) : HAC_ERR_INVALID_ARG;
}
int shac_debug_decode(const shac_format* f, float* nz_dev, void* cuda_stream) {
    return f ? debug_decode(f->f, nz_dev, cuda_stream) : HAC_ERR_INVALID_ARG;
}

int hac_last_launch_count(const hac_format* f) { return f ? f->f.last_launches : 0; }
int shac_last_launch_count(const shac_format* f) { return f ? f->f.last_launches : 0; }

void hac_free(hac_format* f) { delete f; }
void shac_free(shac_format* f) { delete f; }

const char* hac_last_cuda_error(void) { return g_last_cuda_error.c_str(); }

int hac_lost_waits(unsigned int* count) {
    if (!count) return HAC_ERR_INVALID_ARG;
    HAC_CUDA(cudaMemcpyFromSymbol(count, g_lost_waits, sizeof(unsigned int)));
    return HAC_OK;
}

}  // extern "C"
