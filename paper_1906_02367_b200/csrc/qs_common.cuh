// Shared declarations of the sync-round kernels (sm_100a).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/qsparse.h"

namespace qs {

constexpr int MAX_R = 32;            // decode keeps one bit per worker in a 32-bit word
constexpr int GROUP = 128;           // coordinates one warp handles at a time (4 per lane)
constexpr int GPW = 2;               // groups per warp in a tile
constexpr int STILE = 8 * GPW * GROUP;   // coordinates per tile: 8 warps x GPW groups = 2048
constexpr int BLK_TILES = 16;        // tiles per candidate block (32768 coordinates)
constexpr int SUP_BLOCKS = 64;       // blocks per super-block of the two-level candidate counts
#ifndef QS_CHUNK
#define QS_CHUNK 1024
#endif
constexpr int CHUNK = QS_CHUNK;     // candidates per selection chunk (a multiple of the 256 threads)
constexpr int UT_MAX = 2048;         // units whose table fits in the persistent kernel's shared memory
constexpr int U_MAX = 16384;         // units in all: (worker, segment) pairs
constexpr uint32_t ORDER_SUPS_MAX = 2048;   // (worker, super-block) sums the order stage can hold in shared memory
constexpr int UNIT_CAP = 6144;       // candidates of a unit that one block may select from on its own (16 per thread)
constexpr int FB_BINS = 2048;        // bins of the exact fallback histogram (top 11 key bits)
constexpr int FB_SHIFT = 21;
constexpr int FB_CHUNK = 65536;      // coordinates per fallback-histogram block
constexpr uint32_t NO_GUESS = 0xFFFFFFFFu;
constexpr int TRACE_SLOTS = 32;       // time stamps of the persistent kernel's barriers

// cand_q fields
constexpr uint32_t Q_NEG = 1u << 16;
constexpr uint32_t Q_SEL = 1u << 17;

// the local step that precedes a synchronisation: grad R x d, vel R x d or nullptr
struct StepArgs {
    const float* grad;
    float* vel;
    float eta, mu;
};

struct Active {          // workers taking part in a call, ascending
    int n;
    uint32_t bits;
    int r[MAX_R];
};

struct Unit {            // one (worker, segment) pair
    uint32_t tie_t;      // non-zero while a large unit waits for its tie cut: equal keys to keep
    uint32_t spare;
    uint32_t done;       // chunks of the unit that have added their part of the norm (back to 0 after use)
    uint32_t nchunks;
    uint32_t tau;        // sort key of the last kept coordinate
    uint32_t tie_max;    // largest index kept among keys equal to tau
    uint32_t n;          // entries sent (non-zero level)
    float norm;
    uint32_t emin, emax; // exponent range seen by the norm accumulation
};

struct FbBlock {         // fallback histogram work item: one stretch of one segment
    uint32_t seg, start, len;
};

struct Plan {
    int R, nseg, s, sp, qz, bl;
    int wbase, rdiv;           // sharded job: global id of local worker 0, workers in the whole job (divisor of the update)
    uint32_t d, ngroups, ntile, nblk, nsup, K, U, nfb, maxchunks;
    uint32_t seed_lo, seed_hi, round_lo, round_hi;
    uint32_t unit_cap;         // a round whose units all have at most this many candidates selects per block (0: never)
    uint32_t order_sups_max;   // (worker, super-block) pairs up to which the order stage deals its work evenly
    uint32_t spin_limit;       // polls a grid barrier waits before it records QS_TIMEOUT
    int test_miss_barrier;     // test of that path: block 0 stays away from the launch's first barrier
    int block_pack;            // non-zero: every block packs its share before the closing stage (no packing warps beside it)
    uint64_t cap;
    // tables (device)
    const uint32_t* seg_off;   // nseg + 1
    const uint32_t* kseg;      // nseg
    const uint32_t* kprefix;   // nseg + 1
    const uint32_t* grp_seg;   // ngroups: segment of the group's first coordinate
    const uint32_t* target;    // nseg: candidates aimed for
    const uint32_t* seg_order; // nseg: segments by falling candidate target (largest units are dealt first)
    const uint32_t* tile_order; // ntile, or null for 0, 1, 2, ..: the order in which the closing stage hands tiles out (crowded tiles first)
    const float* cscale;       // nseg: fl32(1 / (1 + beta_{k,s}))
    const uint8_t* bidx;       // nseg: bits per index field
    const FbBlock* fb_tab;     // nfb
    // bound state
    float* x; float* xw; float* mem; float* anchors;
    // scratch
    uint32_t* guess;           // R x nseg, sort-key space
    uint32_t* wary;            // R x nseg: rounds for which the unit's prediction still aims wide after a miss
    uint32_t* gap_unit;        // 40 x MAX_R x nseg: per-unit table and gap-length counts of the gap-coded record's two directions
    uint32_t* gap_csum;        // 2 x MAX_R x (K / 1024 + nseg + 1): chunk sums (escapes, index distance) of the gap coder
    uint2* stage;              // R x cap (index, value bits): candidates as the dense pass left them, tile t at t * STILE
    uint32_t* tile_cnt;        // R x (nblk x BLK_TILES): rows padded to whole blocks, the padding stays zero
    uint32_t* blk_count;       // R x nblk, zero between rounds
    uint32_t* sup_count;       // R x nsup, zero between rounds
    uint32_t* seg_start;       // R x (nseg + 1): first candidate of each segment in the ordered list
    uint32_t* fail;            // R
    Unit* units;               // U = R x nseg
    uint32_t* total_chunks;    // 1
    uint32_t* cand_idx;        // R x cap
    float* cand_val;           // R x cap
    uint32_t* cand_key;        // R x cap (Rand_k only)
    uint32_t* cand_q;          // R x cap
    uint32_t* hist;            // 4 x U x 256, zero between rounds
    unsigned long long* eacc;  // U x 256 x 2, zero between rounds
    uint32_t* chunk_cnt;       // maxchunks + 1 (kept | sent << 16 per chunk)
    uint32_t* chunk_dir;       // maxchunks: unit of each chunk, for the packing warps of the closing stage
    uint4* unit_tab;           // U: (start, candidates, first chunk) of each unit, likewise
    uint32_t* gtab;            // 4 (U + 1) + 8 words: the unit table of every block when U > UT_MAX (else null)
    uint32_t* chunk_sel;       // maxchunks + 1 exclusive sums of kept
    uint32_t* chunk_nz;        // maxchunks + 1 exclusive sums of sent
    uint32_t* fb_hist;         // U x FB_BINS, zero between rounds
    uint32_t* sel_idx;         // R x K
    uint32_t* sel_q;           // R x K
    uint32_t* pay_off;         // R x nseg: word offset of the segment's streams (fixed when every kept entry is sent)
    long long* bits;           // R: bits of the worker's record (likewise)
    uint32_t* dec_ent;         // 32 x (nseg + 1): any worker of a sharded job
    uint32_t* dec_pay;         // 32 x nseg
    uint32_t* touch;           // d, zero between rounds: senders of each coordinate (separate master call)
    int* status;
    uint32_t* bar;             // [0] arrivals of the grid barrier, [1] blocks that left the kernel, [2], [3] tile tickets,
                               // [4] unit tickets, [6] chunk tickets of the packing warps
    unsigned long long* trace; // TRACE_SLOTS global-timer stamps of the last persistent launch, or null
    long long* stats;          // device counters: [0] fallback worker-rounds, [1] candidates
};

// ------------------------------------------------------------------ device helpers
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
    for (int i = 0; i < 10; ++i) {
        // each 32 x 32 -> 64-bit product as one wide multiply
        const unsigned long long p0 = (unsigned long long)0xD2511F53u * c.x;
        const unsigned long long p1 = (unsigned long long)0xCD9E8D57u * c.z;
        c = make_uint4((uint32_t)(p1 >> 32) ^ c.y ^ k.x, (uint32_t)p1, (uint32_t)(p0 >> 32) ^ c.w ^ k.y, (uint32_t)p0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}

// the four words for coordinates 4q .. 4q+3 of one worker
__device__ __forceinline__ uint4 philox_quad(const Plan& P, uint32_t worker, uint32_t q,
                                             uint32_t stream) {
    return philox4x32_10(make_uint4(q, worker + (uint32_t)P.wbase, P.round_lo, (P.round_hi << 8) | stream),
                         make_uint2(P.seed_lo, P.seed_hi));
}

__device__ __forceinline__ uint32_t philox_word(const Plan& P, uint32_t worker, uint32_t e,
                                                uint32_t stream) {
    const uint4 o = philox_quad(P, worker, e >> 2, stream);
    const uint32_t j = e & 3u;
    return j == 0 ? o.x : j == 1 ? o.y : j == 2 ? o.z : o.w;
}

__device__ __forceinline__ uint32_t warp_sum(uint32_t v);

// Candidates of one tile, written by the block that just formed u for it (8 warps, warp w owns
// groups GPW w .. GPW w + GPW - 1).  bal[k][j]: ballot of "coordinate 4 lane + j of group k is a
// candidate".  Phase 1 publishes the group counts; after a block-wide barrier phase 2 writes the
// tile's candidates in ascending coordinate order at the tile's fixed place, and the counts.
__device__ __forceinline__ void tile_counts(uint32_t* sh_cnt, int warp, int lane, const uint32_t bal[GPW][4]) {
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < GPW; ++k)
            sh_cnt[warp * GPW + k] = __popc(bal[k][0]) + __popc(bal[k][1]) + __popc(bal[k][2]) + __popc(bal[k][3]);
    }
}

__device__ __forceinline__ void tile_write(const Plan& P, int r, uint32_t tile, const uint32_t* sh_cnt, int warp,
                                           int lane, const uint32_t bal[GPW][4], const float u[GPW][4]) {
    // the last warp owes the tile's total (warp 0 is the one that keeps the copies going); a warp
    // without candidates has nothing else to do
    uint32_t mine = 0;
#pragma unroll
    for (int k = 0; k < GPW; ++k) mine |= bal[k][0] | bal[k][1] | bal[k][2] | bal[k][3];
    if (warp == 7) {
        const uint32_t total = warp_sum(lane < 8 * GPW ? sh_cnt[lane] : 0u);
        if (lane == 0) {
            P.tile_cnt[(size_t)r * P.nblk * BLK_TILES + tile] = total;
            if (total) {
                const uint32_t blk = tile / BLK_TILES;
                atomicAdd(&P.blk_count[(size_t)r * P.nblk + blk], total);
                atomicAdd(&P.sup_count[(size_t)r * P.nsup + blk / SUP_BLOCKS], total);
            }
        }
    }
    if (!mine) return;
    uint32_t base = 0;
    for (int i = 0; i < warp * GPW; ++i) base += sh_cnt[i];
    const size_t off = (size_t)r * P.cap + (size_t)tile * STILE;
    const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
    for (int k = 0; k < GPW; ++k) {
        uint32_t pos = base + __popc(bal[k][0] & lt) + __popc(bal[k][1] & lt) + __popc(bal[k][2] & lt) + __popc(bal[k][3] & lt);
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if ((bal[k][j] >> lane) & 1u) {
                P.stage[off + pos] = make_uint2(tile * (uint32_t)STILE + (uint32_t)((warp * GPW + k) * GROUP + lane * 4 + j),
                                                __float_as_uint(u[k][j]));
                ++pos;
            }
        base += sh_cnt[warp * GPW + k];
    }
}

// Sort key: larger = kept first.  Top_k: |u| bit pattern (shifted up by the spare sign bit);
// Rand_k: complement of the hash, so that the smallest hashes come first.
__device__ __forceinline__ uint32_t topk_key(float u) { return __float_as_uint(u) << 1; }

__device__ __forceinline__ uint32_t warp_sum(uint32_t v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Exclusive scan over the block (blockDim.x a multiple of 32, at most 1024); every thread
// gets the block total too.  sh: 33 words.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* sh, uint32_t* total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const uint32_t incl = warp_incl_scan(v, lane);
    __syncthreads();                       // sh may still be read from a previous call
    if (lane == 31) sh[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        const uint32_t w = lane < nw ? sh[lane] : 0u;
        const uint32_t wi = warp_incl_scan(w, lane);
        sh[lane] = wi - w;
        if (lane == 31) sh[32] = wi;
    }
    __syncthreads();
    *total = sh[32];
    return sh[wid] + incl - v;
}

__device__ __forceinline__ void set_status(const Plan& P, int code) { atomicCAS(P.status, 0, code); }

__host__ __device__ __forceinline__ bool qz_is_sign(int qz) { return qz == QS_SIGN_L1 || qz == QS_SIGN_L2; }
// quantizers that send every kept entry: the streams' places and the bit count never change
__host__ __device__ __forceinline__ bool qz_sends_all(int qz) { return qz_is_sign(qz) || qz == QS_NONE || qz == QS_MINMAX; }
// quantizers whose record has a level stream
__host__ __device__ __forceinline__ bool qz_has_levels(int qz) { return qz == QS_QSGD || qz == QS_QSGD_SCALED || qz == QS_MINMAX; }

__host__ __device__ __forceinline__ uint32_t words_for(uint32_t nfields, uint32_t width) {
    return (uint32_t)(((uint64_t)nfields * width + 31u) >> 5);
}

// words of the streams of a segment that sends n entries, and bits per entry
__host__ __device__ __forceinline__ uint32_t streams_words(uint32_t n, uint32_t bi, uint32_t bl, int qz) {
    if (qz == QS_NONE) return words_for(n, bi) + n;                     // indices, then 32-bit values
    if (qz == QS_MINMAX) return words_for(n, bi) + words_for(n, bl);    // indices, then levels (no signs)
    return words_for(n, bi) + words_for(n, 1) + (!qz_is_sign(qz) ? words_for(n, bl) : 0u);
}
__host__ __device__ __forceinline__ uint32_t entry_bits(uint32_t bi, uint32_t bl, int qz) {
    if (qz == QS_NONE) return bi + 32u;
    if (qz == QS_MINMAX) return bi + bl;
    return bi + 1u + (!qz_is_sign(qz) ? bl : 0u);
}

// fp32 level of the QSGD quantizer and the value it stands for
__device__ __forceinline__ int qsgd_level(float u, float N, int s, uint32_t w) {
    if (N == 0.0f) return 0;
    const float a = fabsf(u) * (float)s;
    const float p = a / N;
    const float l = floorf(p);
    const float f = p - l;
    const float U = (float)(w >> 8) * 5.9604644775390625e-08f;
    const int level = (int)l + (U < f ? 1 : 0);
    return level < s ? level : s;
}

// The min/max quantizer: smallest and largest kept value travel as ordered 32-bit keys (larger
// float = larger key), which atomicMin / atomicMax can work on.
__device__ __forceinline__ uint32_t float_order(float v) {
    const uint32_t b = __float_as_uint(v);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float order_float(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
// level 1 .. s of the min/max quantizer (level l stands for lo + (l - 1) D) and the value
__device__ __forceinline__ int minmax_level(float v, float lo, float hi, int s, uint32_t w) {
    const float D = (hi - lo) / (float)(s - 1);
    if (!(D > 0.0f)) return 1;
    const float p = (v - lo) / D;
    const float l = floorf(p);
    const float f = p - l;
    const float U = (float)(w >> 8) * 5.9604644775390625e-08f;
    int j = (int)l + (U < f ? 1 : 0);
    j = j < 0 ? 0 : j;
    j = j > s - 1 ? s - 1 : j;
    return j + 1;
}
__device__ __forceinline__ float minmax_value(float lo, float hi, int s, int level) {
    const float D = (hi - lo) / (float)(s - 1);
    const float step = (float)(level - 1) * D;
    return lo + step;
}

__device__ __forceinline__ float coord_value(const Plan& P, float N, int level, bool neg, float c,
                                             uint32_t k) {
    float g;
    if (qz_is_sign(P.qz)) {                      // Lemma 3: the l1 (m = 1) or l2 (m = 2) norm over k
        g = N / (float)k;
    } else {
        g = (N * (float)level) / (float)P.s;
        if (P.qz == QS_QSGD_SCALED) g = g * c;
    }
    return neg ? -g : g;
}

}  // namespace qs
