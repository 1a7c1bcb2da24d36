// Internal definitions shared by the host builder (hac_build.cpp) and the device side
// (hac_kernels.cu) of the library.  Not part of the public boundary.
#pragma once

#include <cstddef>
#include <cstdint>
#include <string>
#include <vector>

#include "hac.h"

namespace hacb200 {

constexpr int kMaxCodeLen = 32;
constexpr int kLutBitsMax = 12;          // full-width decode table: 2^L entries of 16 bits (12-bit rank, 4-bit length)
static_assert(kLutBitsMax < 16 && HAC_MAX_SYMBOLS <= 4096, "a table entry holds (rank << 4) | length in 16 bits");
constexpr int kL1BitsMax = 10;           // level-1 table of the kernels: 2^L1 entries of 8 bytes
constexpr int kSubBitsMax = 8;           // widest level-2 sub-table
constexpr int kXtMantMax = 5;            // magnitude table: at most 32 << 5 entries (the size of the prefix table)

// Index of a 32-bit window into the magnitude table with `mant` mantissa bits (see DecodeTables::xt).
inline uint32_t xt_index(uint32_t window, int mant) {
    const uint32_t u = ~window | 1u;
    int e = 31;
    while (!(u >> e)) --e;
    const uint32_t norm = u << (31 - e);                     // leading one at bit 31
    const uint32_t frac = mant ? ((norm << 1) >> (32 - mant)) : 0u;
    return ((uint32_t)e << mant) | frac;
}
constexpr size_t kSubTableBytesMax = 24 * 1024;
constexpr int kStreamSlackWords = 4;     // zero words after the stream (decoder reads ahead)
constexpr size_t kTaskOffBytesMax = (size_t)64 << 20;
constexpr int kItemWords = 48;           // sHAC work item record: 12 header words, 2 x 16 words of sub-segment bit lengths, 4 spare

// Decoding tables derived from the code lengths (canonical Huffman).  "rank" is the position of
// a symbol in (length, id) order; values are stored in rank order so that short, frequent code
// words use the first entries.
struct DecodeTables {
    int lut_bits = 0;                         // L = min(max_len, kLutBitsMax)
    std::vector<uint16_t> lut;                // [2^L] (rank << 4) | len, 0 = code longer than L
    std::vector<float> rank_value;            // [k_eff]
    std::vector<uint16_t> rank_symbol;        // [k_eff] symbol id of each rank
    // Two-level table used by the kernels.  l1[i] for the L1-bit prefix i is {value bits, length}
    // when the code word ends within the prefix, else {byte offset of a sub-table, 0x80000000 | b}:
    // the sub-table is indexed by the next b bits and holds {value bits, length} or {0, 0} (code
    // word longer than L1 + b: found by the search over lengths).
    int l1_bits = 0;
    std::vector<uint32_t> l1;                 // [2^l1_bits * 2]
    std::vector<uint32_t> sub;                // [entries * 2]
    // Zero-run variant of l1 (HAC with a short code word for 0): an entry covers as many zero symbols
    // as fit in the prefix plus, if it fits too, the non-zero symbol after them:
    // {value bits of that symbol (0 if none), length | (symbols covered << 8)}; prefixes of longer code
    // words keep their sub-table entry.  Empty when the format has no use for it.
    std::vector<uint32_t> l1_runs;            // [2^l1_bits * 2]
    uint32_t zero_len = 0;                    // code length of the zero symbol (0 = none)
    // Table indexed by magnitude instead of by prefix.  A canonical code puts its long code words at
    // the top of the code space (many leading ones), where a prefix table is far too coarse, and its
    // short ones at the bottom, where it is finer than needed.  With u = ~window | 1 (32 bits), the
    // index is the exponent of u (31 - leading ones of the window) followed by the xt_mant bits after
    // its leading one: exactly the top bits of u converted to float with rounding toward zero, biased
    // exponent 127 removed.  A cell that lies inside one code word's range holds {value bits, length};
    // any other cell holds {0, 0x80000000} (found by the search over lengths).  32 << xt_mant entries.
    // Built when code words are longer than the prefix table; used when it leaves fewer symbols
    // unresolved than the prefix table does.
    int xt_mant = -1;                         // -1: not built
    std::vector<uint32_t> xt;                 // [(32 << xt_mant) * 2]
    double xt_unresolved = 0.0;               // share of the symbols the magnitude table leaves to the search
    double l1_unresolved = 0.0;               // share of the symbols whose code word is longer than l1_bits
    bool use_xt = false;
    uint64_t limit[kMaxCodeLen + 2] = {};     // left-aligned (32-bit) end of the codes of length l
    uint32_t first_left[kMaxCodeLen + 2] = {};// left-aligned first code of length l
    uint32_t rank_base[kMaxCodeLen + 2] = {}; // rank of the first code of length l
};

struct uint2_host { uint32_t x, y; };

// Pointers into the device image, filled by upload/attach.
struct DeviceImage {
    void* base = nullptr;
    size_t bytes = 0;
    const uint32_t* stream = nullptr;
    const uint16_t* lut = nullptr;
    const uint2_host* l1 = nullptr;
    const uint2_host* sub = nullptr;
    const uint2_host* l1_runs = nullptr;
    const uint2_host* xt = nullptr;
    const float* rank_value = nullptr;
    const uint64_t* limit = nullptr;          // [34]
    const uint32_t* first_left = nullptr;     // [34]
    const uint32_t* rank_base = nullptr;      // [34]
    const uint64_t* seg_bit_off = nullptr;
    const uint16_t* sub_bits = nullptr;
    const uint32_t* seg_col = nullptr;
    const uint32_t* seg_first = nullptr;
    const void* ri = nullptr;
    const uint32_t* cb = nullptr;
    const void* unit_info = nullptr;
    const uint64_t* task_off = nullptr;
    const uint32_t* task_pos = nullptr;
};

struct Format {
    bool sparse = false;                      // sHAC
    int64_t n = 0, m = 0;
    int64_t nnz = 0;                          // entries surviving pruning
    int64_t symbols = 0;                      // n*m (HAC) or nnz (sHAC)
    uint32_t S = 0;                           // symbols per sub-segment
    uint32_t G = 0;                           // HAC: segments per column
    uint32_t ri_bits = 0;
    // alphabet
    std::vector<float> codebook;              // ascending
    std::vector<uint8_t> code_len;
    std::vector<uint32_t> codes;
    std::vector<int64_t> counts;
    uint32_t max_len = 0, min_len = 0;
    // stream
    std::vector<uint32_t> stream;             // stream_words data words + pad words
    int64_t stream_bits = 0, stream_words = 0, pad_words = 0;
    // sHAC
    std::vector<uint16_t> ri16;
    std::vector<uint32_t> ri32;
    std::vector<uint32_t> cb;
    // offset index
    std::vector<uint64_t> seg_bit_off;
    std::vector<uint16_t> sub_bits;
    std::vector<uint32_t> seg_first, seg_col;
    std::vector<uint32_t> item_info;          // sHAC, device only: kItemWords words per work item (see ShacItem)
    // HAC, device only: start bit of every sub-segment of every column, [ceil(n/S) + 1][m] (the last row
    // holds the columns' ends), for the batched kernel, whose lanes are columns.  Left empty, and then
    // derived from the offset index on every call, when it would exceed kTaskOffBytesMax.
    std::vector<uint64_t> task_off;
    // sHAC, device only, for the batched tensor-core kernel: the rows are cut into tasks of tc_rows rows (a
    // power of two chosen so that a task of a column holds a few dozen stored entries); task_off[t][j] is
    // the bit where the first entry of column j with row >= t * tc_rows starts and task_pos[t][j] its
    // position in nz / ri ([tasks + 1][m]; the last row holds the columns' ends).  Empty (no tensor-core
    // path) when the tables would exceed kTaskOffBytesMax.
    std::vector<uint32_t> task_pos;
    uint32_t tc_rows = 0;
    uint32_t max_task_chunks = 1;             // largest 16-byte span of the stream a task of a column covers
    uint32_t max_task_ri_chunks = 1;          // the same for its slice of ri
    uint32_t max_unit_chunks = 0;             // largest 16-byte span a segment's stream covers
    uint32_t max_sub_chunks = 0;              // same for a single sub-segment
    uint32_t max_units_per_col = 0;
    bool has_empty_col = false;
    // derived
    DecodeTables tables;
    DeviceImage dev;
    mutable int last_launches = 0;
    // epilogue of the product being launched (set by the *_dot_layer entry points for the duration of a call)
    mutable const float* epi_bias = nullptr;
    mutable uint32_t epi_relu = 0;
};

int build_impl(const float* W, int64_t n, int64_t m, int64_t ldw, const hac_build_params* p,
               bool sparse, Format& f);
void make_decode_tables(Format& f);
int decode_on_host(const Format& f, float* Wq, int64_t ldq);
void fill_size_report(const Format& f, hac_size_report* r);

// device image layout: offsets of every section (256-byte aligned), total size
struct ImageLayout {
    size_t stream, lut, l1, sub, l1_runs, xt, rank_value, limit, first_left, rank_base, seg_bit_off, sub_bits, seg_col,
        seg_first, ri, cb, unit_info, task_off, task_pos, total;
};
ImageLayout image_layout(const Format& f);

// Text that hac_last_cuda_error() returns on this thread (set by every file that makes CUDA calls).
void set_last_cuda_error(const std::string& text);

}  // namespace hacb200

struct hac_format { hacb200::Format f; };
struct shac_format { hacb200::Format f; };
