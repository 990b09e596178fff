// C boundary of the sync-round library: context, tables, scratch and the order of launches.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <string>
#include <vector>

#include "qs_kernels.h"

using namespace qs;

struct qs_ctx {
    Plan P;
    cudaStream_t st;
    int sms, mid_grid;
    bool bound, aligned, compressed, use_tma;
    Active last;                       // workers of the last compression
    std::vector<int64_t> off, kseg;    // host copies of the segment table
    int64_t wire_words, gap_words;
    uint32_t longest_k, most_words, row_chunks;   // of the gap-coded record: largest k_seg, most stream words of a segment, chunk sums per worker
    uint64_t round;
    int64_t launches, rounds;
    std::string err;
    std::vector<void*> owned;          // everything cudaMalloc'ed for the current tables
    // optional per-phase timing of qs_sync_round (events on the context's stream)
    bool timing;
    std::vector<cudaEvent_t> ev;       // TIMING_ROUNDS x TIMING_MARKS
    int ev_used;
    double phase_ms[2];
    int64_t timed_rounds;
};

namespace {

constexpr int TIMING_MARKS = 3, TIMING_ROUNDS = 512;

void mark(qs_ctx* c, int slot) {
    if (c->timing) cudaEventRecord(c->ev[(size_t)c->ev_used * TIMING_MARKS + slot], c->st);
}

// adds the recorded rounds to the per-phase sums (synchronises the stream)
void fold_timing(qs_ctx* c) {
    if (!c->ev_used) return;
    cudaStreamSynchronize(c->st);
    for (int i = 0; i < c->ev_used; ++i)
        for (int ph = 0; ph < TIMING_MARKS - 1; ++ph) {
            float ms = 0.0f;
            if (cudaEventElapsedTime(&ms, c->ev[(size_t)i * TIMING_MARKS + ph], c->ev[(size_t)i * TIMING_MARKS + ph + 1]) == cudaSuccess)
                c->phase_ms[ph] += ms;
        }
    c->timed_rounds += c->ev_used;
    c->ev_used = 0;
}

int fail(qs_ctx* c, int code, const char* what) {
    if (c) c->err = what;
    return code;
}

int cuda_fail(qs_ctx* c, cudaError_t e, const char* where) {
    if (c) c->err = std::string(where) + ": " + cudaGetErrorString(e);
    return QS_CUDA;
}

#define QS_CUDA_TRY(ctx, call)                                  \
    do {                                                        \
        cudaError_t e_ = (call);                                \
        if (e_ != cudaSuccess) return cuda_fail(ctx, e_, #call); \
    } while (0)

int after_launch(qs_ctx* c, int kernels, const char* where) {
    c->launches += kernels;
    cudaError_t e = cudaPeekAtLastError();
    if (e != cudaSuccess) return cuda_fail(c, e, where);
    return QS_OK;
}

void release(qs_ctx* c) {
    for (void* p : c->owned) cudaFree(p);
    c->owned.clear();
}

template <class T>
int dev_alloc(qs_ctx* c, T** out, size_t count, bool zero) {
    void* p = nullptr;
    const size_t bytes = (count ? count : 1) * sizeof(T);
    if (cudaMalloc(&p, bytes) != cudaSuccess) {
        cudaGetLastError();
        return fail(c, QS_ALLOC, "scratch allocation failed");
    }
    c->owned.push_back(p);
    if (zero && cudaMemsetAsync(p, 0, bytes, c->st) != cudaSuccess) return fail(c, QS_CUDA, "memset failed");
    *out = static_cast<T*>(p);
    return QS_OK;
}

template <class T>
int dev_upload(qs_ctx* c, const T** out, const std::vector<T>& host) {
    T* p = nullptr;
    int rc = dev_alloc(c, &p, host.size(), false);
    if (rc != QS_OK) return rc;
    if (!host.empty())
        QS_CUDA_TRY(c, cudaMemcpyAsync(p, host.data(), host.size() * sizeof(T), cudaMemcpyHostToDevice, c->st));
    *out = p;
    return QS_OK;
}

int ceil_log2(uint64_t v) {
    int b = 0;
    while ((1ull << b) < v) ++b;
    return b;
}

// candidates aimed for in a segment of n coordinates keeping k
uint32_t candidate_target(int sp, uint64_t n, uint64_t k) {
    double slack;
    if (sp == QS_RANDK) {
        slack = 6.0 * std::sqrt((double)k) + 32.0;           // the hash is uniform: binomial spread
    } else {
        const double ratio = (double)k / (double)n;
        const double frac = ratio <= 0.02 ? 0.5 : 0.25;
        slack = std::fmax(std::fmax(frac * (double)k, 16.0 * std::sqrt((double)k)), 16.0);
    }
    const double t = (double)k + slack;
    return (uint32_t)(t >= (double)n ? n : (uint64_t)t);
}

int make_active(const qs_ctx* c, const uint8_t* mask, Active* a) {
    a->n = 0;
    a->bits = 0;
    for (int r = 0; r < c->P.R; ++r)
        if (!mask || mask[r]) {
            a->r[a->n++] = r;
            a->bits |= 1u << r;
        }
    return a->n;
}

// the records to decode: workers of the whole (possibly sharded) job
int make_active_job(const qs_ctx* c, const uint8_t* mask, Active* a) {
    a->n = 0;
    a->bits = 0;
    for (int r = 0; r < c->P.rdiv; ++r)
        if (!mask || mask[r]) {
            a->r[a->n++] = r;
            a->bits |= 1u << r;
        }
    return a->n;
}

int install_segments(qs_ctx* c, int nseg, const int64_t* offsets, const int64_t* kseg) {
    Plan& P = c->P;
    const int64_t d = (int64_t)P.d;
    if (nseg < 1 || !offsets || !kseg || offsets[0] != 0 || offsets[nseg] != d)
        return fail(c, QS_INVALID_ARG, "segments must start at 0 and end at d");
    if ((int64_t)P.R * nseg > U_MAX) return fail(c, QS_INVALID_ARG, "R x nseg exceeds 16384 units");
    for (int g = 0; g < nseg; ++g) {
        const int64_t n = offsets[g + 1] - offsets[g];
        if (n < 1 || kseg[g] < 1 || kseg[g] > n) return fail(c, QS_INVALID_ARG, "need 1 <= k_seg <= segment length");
    }
    QS_CUDA_TRY(c, cudaStreamSynchronize(c->st));
    release(c);
    c->off.assign(offsets, offsets + nseg + 1);
    c->kseg.assign(kseg, kseg + nseg);
    c->compressed = false;

    const int R = P.R;
    P.nseg = nseg;
    P.U = (uint32_t)R * nseg;
    P.ngroups = (uint32_t)((d + GROUP - 1) / GROUP);
    P.ntile = (uint32_t)((d + STILE - 1) / STILE);
    P.nblk = (P.ntile + BLK_TILES - 1) / BLK_TILES;
    P.nsup = (P.nblk + SUP_BLOCKS - 1) / SUP_BLOCKS;
    P.cap = (uint64_t)d;
    P.bl = std::max(1, ceil_log2((uint64_t)P.s));
    P.maxchunks = (uint32_t)R * (uint32_t)((d + CHUNK - 1) / CHUNK + nseg);

    std::vector<uint32_t> h_off(nseg + 1), h_k(nseg), h_kp(nseg + 1, 0), h_target(nseg), h_grp, h_guess, h_order(nseg);
    std::vector<uint32_t> h_pay((size_t)R * nseg, 0u);
    std::vector<long long> h_bits(R, 0ll);
    std::vector<float> h_c(nseg);
    std::vector<uint8_t> h_bi(nseg);
    std::vector<FbBlock> h_fb;
    int64_t words = 2 * (int64_t)nseg;
    for (int g = 0; g < nseg; ++g) {
        const uint64_t n = (uint64_t)(offsets[g + 1] - offsets[g]), k = (uint64_t)kseg[g];
        h_off[g] = (uint32_t)offsets[g];
        h_k[g] = (uint32_t)k;
        h_kp[g + 1] = h_kp[g] + (uint32_t)k;
        h_target[g] = candidate_target(P.sp, n, k);
        const double a = (double)k / ((double)P.s * (double)P.s), b = std::sqrt((double)k) / (double)P.s;
        h_c[g] = (float)(1.0 / (1.0 + (a < b ? a : b)));
        h_bi[g] = (uint8_t)std::max(1, ceil_log2(n));
        // quantizers that send every kept entry: the streams' places and the bit count never change
        if (qz_sends_all(P.qz))
            for (int r = 0; r < R; ++r) {
                h_pay[(size_t)r * nseg + g] = (uint32_t)words;
                h_bits[r] += 64 + (long long)k * entry_bits(h_bi[g], (uint32_t)P.bl, P.qz);
            }
        words += streams_words((uint32_t)k, h_bi[g], (uint32_t)P.bl, P.qz);
        h_order[g] = (uint32_t)g;
        for (uint64_t s0 = 0; s0 < n; s0 += FB_CHUNK)
            h_fb.push_back(FbBlock{(uint32_t)g, (uint32_t)(offsets[g] + s0), (uint32_t)std::min<uint64_t>(FB_CHUNK, n - s0)});
    }
    h_off[nseg] = (uint32_t)d;
    std::stable_sort(h_order.begin(), h_order.end(), [&](uint32_t a, uint32_t b) { return h_target[a] > h_target[b]; });
    P.K = h_kp[nseg];
    P.nfb = (uint32_t)h_fb.size();
    c->wire_words = words;
    {
        int64_t gw = 5 * (int64_t)nseg;
        uint64_t longest = 0, most = 0;
        for (int g = 0; g < nseg; ++g) {
            const uint32_t k = (uint32_t)kseg[g];
            const uint64_t all = streams_words(k, h_bi[g], (uint32_t)P.bl, P.qz);
            // fields and exceptions together never exceed (k - 1) b_idx bits; two streams, each padded to a word
            gw += (int64_t)words_for(k - 1, h_bi[g]) + 1 + (int64_t)all - (int64_t)words_for(k, h_bi[g]);
            longest = std::max<uint64_t>(longest, k);
            most = std::max<uint64_t>(most, all);
        }
        c->gap_words = gw;
        c->longest_k = (uint32_t)longest;
        c->most_words = (uint32_t)most;
        c->row_chunks = (uint32_t)(P.K / gap_chunk()) + (uint32_t)nseg + 1u;
    }
    if (nseg > 1) {
        h_grp.resize((size_t)P.ntile * (STILE / GROUP));     // whole tiles: the dense pass copies a tile's entries at once
        int sg = 0;
        for (uint32_t g = 0; g < (uint32_t)h_grp.size(); ++g) {
            const int64_t e = (int64_t)g * GROUP;
            while (sg + 1 < nseg && e >= offsets[sg + 1]) ++sg;
            h_grp[g] = (uint32_t)sg;
        }
    }
    // Tiles in which the workers together keep more entries than there are coordinates (small
    // tensors kept whole, Section 5.1's k_t = min(d_t, 1000)) cost one warp of the closing stage
    // many times an ordinary tile: they are handed out first, so that the rest of the stage hides them.
    std::vector<uint32_t> h_tiles;
    {
        std::vector<double> crowd(P.ntile, 0.0);
        bool any = false;
        for (int g = 0; g < nseg; ++g) {
            const int64_t n = offsets[g + 1] - offsets[g];
            const double per = (double)R * (double)std::min<uint64_t>(h_target[g], (uint64_t)n) / (double)n;
            if (per < 0.25) continue;                              // (ordinary ratios: never crowded)
            for (int64_t t = offsets[g] / STILE; t * STILE < offsets[g + 1]; ++t) {
                const int64_t a = std::max<int64_t>(offsets[g], t * STILE), b = std::min<int64_t>(offsets[g + 1], (t + 1) * STILE);
                crowd[t] += per * (double)(b - a);
            }
        }
        std::vector<uint32_t> heavy, rest;
        for (uint32_t t = 0; t < P.ntile; ++t) (crowd[t] > 1024.0 ? heavy : rest).push_back(t);
        any = !heavy.empty();
        if (any) {
            std::stable_sort(heavy.begin(), heavy.end(), [&](uint32_t a, uint32_t b) { return crowd[a] > crowd[b]; });
            // every eighth place at the front: a block draws a handful of tiles when it starts, and
            // should get one crowded tile among them, not all of them
            const size_t gap = heavy.size() * 8 <= P.ntile ? 8 : 1;
            size_t ih = 0, ir = 0;
            h_tiles.resize(P.ntile);
            for (size_t t = 0; t < P.ntile; ++t)
                h_tiles[t] = (ih < heavy.size() && (t % gap == 0 || ir == rest.size())) ? heavy[ih++] : rest[ir++];
        }
    }
    // first prediction: none for Top_k (the first round takes the exact pass); for Rand_k the
    // hash is uniform, so the cut that lets `target` coordinates through is known in advance
    h_guess.assign((size_t)R * nseg, NO_GUESS);
    if (P.sp == QS_RANDK)
        for (int r = 0; r < R; ++r)
            for (int g = 0; g < nseg; ++g) {
                const uint64_t n = (uint64_t)(offsets[g + 1] - offsets[g]);
                const uint64_t cut = h_target[g] >= n ? 0xffffffffull
                                                      : std::min<uint64_t>(0xffffffffull, ((uint64_t)h_target[g] << 32) / n);
                h_guess[(size_t)r * nseg + g] = ~(uint32_t)cut;
            }

    int rc;
#define UP(field, vec) if ((rc = dev_upload(c, &P.field, vec)) != QS_OK) return rc
    UP(seg_off, h_off); UP(kseg, h_k); UP(kprefix, h_kp); UP(grp_seg, h_grp); UP(target, h_target);
    UP(cscale, h_c); UP(bidx, h_bi); UP(fb_tab, h_fb); UP(seg_order, h_order);
    P.tile_order = nullptr;
    if (!h_tiles.empty()) UP(tile_order, h_tiles);
#undef UP
    const uint32_t* g_up = nullptr;
    if ((rc = dev_upload(c, &g_up, h_guess)) != QS_OK) return rc;
    P.guess = const_cast<uint32_t*>(g_up);
#define AL(field, count, zero) if ((rc = dev_alloc(c, &P.field, (size_t)(count), zero)) != QS_OK) return rc
    AL(wary, P.U, true);
    AL(gap_unit, (size_t)gap_unit_words() * MAX_R * nseg, true);
    AL(gap_csum, (size_t)2 * MAX_R * c->row_chunks, true);
    AL(stage, (size_t)R * P.cap, false);
    AL(tile_cnt, (size_t)R * P.nblk * BLK_TILES, true);
    AL(blk_count, (size_t)R * P.nblk, true);
    AL(sup_count, (size_t)R * P.nsup, true);
    AL(seg_start, (size_t)R * (nseg + 1), true);
    AL(fail, R, true);
    AL(units, P.U, true);
    AL(total_chunks, 1, true);
    AL(cand_idx, (size_t)R * P.cap, false);
    AL(cand_val, (size_t)R * P.cap, false);
    AL(cand_q, (size_t)R * P.cap, false);
    if (P.sp == QS_RANDK) { AL(cand_key, (size_t)R * P.cap, false); } else P.cand_key = nullptr;
    AL(hist, (size_t)4 * P.U * 256, true);
    AL(eacc, (size_t)P.U * 256 * 2, true);
    AL(chunk_cnt, (size_t)P.maxchunks + 1, true);
    AL(chunk_dir, (size_t)P.maxchunks + 1, false);
    AL(unit_tab, P.U, false);
    if (P.U > (uint32_t)UT_MAX) { AL(gtab, (size_t)4 * (P.U + 1) + 8, true); } else P.gtab = nullptr;
    AL(chunk_sel, (size_t)P.maxchunks + 1, true);
    AL(chunk_nz, (size_t)P.maxchunks + 1, true);
    AL(fb_hist, (size_t)P.U * FB_BINS, true);
    AL(sel_idx, (size_t)R * P.K, true);
    AL(sel_q, (size_t)R * P.K, true);
    AL(pay_off, P.U, false);
    AL(bits, R, false);
    QS_CUDA_TRY(c, cudaMemcpyAsync(P.pay_off, h_pay.data(), h_pay.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, c->st));
    QS_CUDA_TRY(c, cudaMemcpyAsync(P.bits, h_bits.data(), h_bits.size() * sizeof(long long), cudaMemcpyHostToDevice, c->st));
    AL(dec_ent, (size_t)32 * (nseg + 1), true);
    AL(dec_pay, (size_t)32 * nseg, true);
    AL(touch, (size_t)d, true);
    AL(status, 1, true);
    AL(bar, 8, true);
    AL(trace, TRACE_SLOTS, true);
    AL(stats, 2, true);
#undef AL
    QS_CUDA_TRY(c, cudaStreamSynchronize(c->st));
    return QS_OK;
}

// scratch that must be zero when a round starts; restored after a device-side error
int rezero(qs_ctx* c) {
    Plan& P = c->P;
    QS_CUDA_TRY(c, cudaMemsetAsync(P.hist, 0, sizeof(uint32_t) * 4 * P.U * 256, c->st));
    QS_CUDA_TRY(c, cudaMemsetAsync(P.eacc, 0, sizeof(unsigned long long) * P.U * 256 * 2, c->st));
    QS_CUDA_TRY(c, cudaMemsetAsync(P.fb_hist, 0, sizeof(uint32_t) * P.U * FB_BINS, c->st));
    QS_CUDA_TRY(c, cudaMemsetAsync(P.touch, 0, sizeof(uint32_t) * P.d, c->st));
    QS_CUDA_TRY(c, cudaMemsetAsync(P.fail, 0, sizeof(uint32_t) * P.R, c->st));
    QS_CUDA_TRY(c, cudaMemsetAsync(P.units, 0, sizeof(Unit) * P.U, c->st));
    QS_CUDA_TRY(c, cudaMemsetAsync(P.status, 0, sizeof(int), c->st));
    QS_CUDA_TRY(c, cudaMemsetAsync(P.bar, 0, 8 * sizeof(uint32_t), c->st));
    QS_CUDA_TRY(c, cudaMemsetAsync(P.blk_count, 0, sizeof(uint32_t) * P.R * P.nblk, c->st));
    QS_CUDA_TRY(c, cudaMemsetAsync(P.sup_count, 0, sizeof(uint32_t) * P.R * P.nsup, c->st));
    return QS_OK;
}

uint64_t take_round(qs_ctx* c, uint64_t round) {
    if (round == QS_ROUND_AUTO) return c->round++;
    c->round = round + 1;
    return round;
}

int run_mid(qs_ctx* c, const Active& act, int do_compress, int do_pack, int do_decode, int do_broadcast,
            uint32_t* wire, int64_t stride, int64_t* bits_out) {
    const cudaError_t e = launch_mid(c->P, act, do_compress, do_pack, do_decode, do_broadcast, c->aligned ? 1 : 0,
                                     wire, stride, (long long)c->wire_words, (long long*)bits_out, c->mid_grid, c->st);
    c->P.test_miss_barrier = 0;                    // the test of the bounded wait concerns one launch
    if (e != cudaSuccess) return cuda_fail(c, e, "persistent kernel");
    return after_launch(c, 1, "persistent kernel");
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// dense pass, then the persistent kernel for the stages asked for
int round_body(qs_ctx* c, uint64_t round, const Active& act, bool fused, uint32_t* wire, int64_t stride,
               int64_t* bits_out, const StepArgs* step = nullptr) {
    Plan& P = c->P;
    P.round_lo = (uint32_t)round;
    P.round_hi = (uint32_t)(round >> 32);
    int rc;
    if (fused) mark(c, 0);
    StepArgs sa = {nullptr, nullptr, 0.0f, 0.0f};
    int kind = 0;                                // local step taken inside the dense pass: 0 none, 1 plain, 2 momentum
    if (step) {
        sa = *step;
        const bool rows16 = c->aligned && aligned16(sa.grad) && aligned16(sa.vel);
        if (c->use_tma && rows16 && pass_a_tma_usable(P, true, sa.vel ? 2 : 1)) {
            kind = sa.vel ? 2 : 1;
        } else {                                 // the step as a launch of its own, then the plain dense pass
            launch_local_step(P, act, sa, rows16, c->sms, c->st);
            if ((rc = after_launch(c, 1, "local_step")) != QS_OK) return rc;
        }
    }
    if (c->use_tma && pass_a_tma_usable(P, c->aligned, kind)) {
        const cudaError_t e = launch_pass_a_tma(P, act, sa, kind, c->sms, c->st);
        if (e != cudaSuccess) return cuda_fail(c, e, "pass_a (bulk copy)");
    } else {
        launch_pass_a(P, act, 0, c->aligned, c->sms, c->st);
    }
    if ((rc = after_launch(c, 1, "pass_a")) != QS_OK) return rc;
    if (fused) {
        mark(c, 1);
    }
    rc = run_mid(c, act, 1, fused, fused, fused, wire, stride, bits_out);
    if (fused) {
        mark(c, 2);
        if (c->timing && ++c->ev_used == TIMING_ROUNDS) fold_timing(c);
    }
    if (rc != QS_OK) return rc;
    c->last = act;
    c->compressed = true;
    c->rounds += 1;
    return QS_OK;
}

}  // namespace

extern "C" {

int qs_init(qs_ctx** out, int R, int64_t d, int64_t k, int s, int op, uint64_t seed, void* cuda_stream) {
    if (!out) return QS_INVALID_ARG;
    *out = nullptr;
    const int sp = op & 15, qz = op >> 4;
    if (R < 1 || R > MAX_R || d < 1 || d > (1ll << 32) - 4096 || k < 1 || k > d || s < 1 || s > 65535) return QS_INVALID_ARG;   // (32-bit tile arithmetic on the device)
    if ((sp != QS_TOPK && sp != QS_RANDK) || (qz != QS_QSGD && qz != QS_QSGD_SCALED && qz != QS_SIGN_L1 && qz != QS_NONE && qz != QS_SIGN_L2 && qz != QS_MINMAX)) return QS_INVALID_ARG;
    if (qz == QS_MINMAX && s < 2) return QS_INVALID_ARG;      // two levels at least: the smallest and the largest entry
    qs_ctx* c = new qs_ctx();
    std::memset(&c->P, 0, sizeof(Plan));
    c->st = static_cast<cudaStream_t>(cuda_stream);
    c->bound = c->aligned = c->compressed = false;
    c->use_tma = std::getenv("QSPARSE_NO_TMA") == nullptr;
    c->round = 0;
    c->launches = c->rounds = 0;
    c->wire_words = 0;
    c->timing = false;
    c->ev_used = 0;
    c->timed_rounds = 0;
    for (double& a : c->phase_ms) a = 0.0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        delete c;
        return QS_CUDA;
    }
    const int per_sm = mid_blocks_per_sm(sp == QS_RANDK);
    if (per_sm < 1) { delete c; return QS_CUDA; }
    int want = 4;                                  // blocks of the persistent kernel per SM
    if (const char* e = std::getenv("QSPARSE_MID_PER_SM")) want = std::atoi(e) > 0 ? std::atoi(e) : want;
    c->mid_grid = c->sms * (per_sm < want ? per_sm : want);
    Plan& P = c->P;
    P.R = R; P.d = (uint32_t)d; P.s = s; P.sp = sp; P.qz = qz;
    P.wbase = 0; P.rdiv = R;
    P.unit_cap = UNIT_CAP;                         // QSPARSE_UNIT_CAP (0 .. 4096) overrides, for tests of both paths
    if (const char* e = std::getenv("QSPARSE_UNIT_CAP")) P.unit_cap = (uint32_t)std::min(std::max(std::atoi(e), 0), UNIT_CAP);
    P.order_sups_max = ORDER_SUPS_MAX;             // QSPARSE_ORDER_EVEN_MAX (0 .. 2048) overrides, for tests of both order stages
    if (const char* e = std::getenv("QSPARSE_ORDER_EVEN_MAX")) P.order_sups_max = (uint32_t)std::min(std::max(std::atoi(e), 0), (int)ORDER_SUPS_MAX);
    P.block_pack = std::getenv("QSPARSE_BLOCK_PACK") != nullptr;   // for tests of both ways of packing in a whole round
    P.spin_limit = 1u << 22;                       // barrier polls before giving up (about a second)
    if (const char* e = std::getenv("QSPARSE_SPIN_LIMIT")) P.spin_limit = (uint32_t)std::max(std::atoi(e), 16);
    P.test_miss_barrier = std::getenv("QSPARSE_TEST_MISS_BARRIER") != nullptr;   // one launch only, see run_mid
    P.seed_lo = (uint32_t)seed; P.seed_hi = (uint32_t)(seed >> 32);
    const int64_t offsets[2] = {0, d};
    const int rc = install_segments(c, 1, offsets, &k);
    if (rc != QS_OK) { release(c); delete c; return rc; }
    *out = c;
    return QS_OK;
}

int qs_set_segments(qs_ctx* c, int nseg, const int64_t* offsets, const int64_t* k_seg) {
    if (!c) return QS_INVALID_ARG;
    return install_segments(c, nseg, offsets, k_seg);
}

int qs_bind(qs_ctx* c, float* x, float* xw, float* mem, float* anchors) {
    if (!c || !x || !xw || !mem) return fail(c, QS_INVALID_ARG, "x, xw and mem are required");
    c->P.x = x; c->P.xw = xw; c->P.mem = mem; c->P.anchors = anchors;
    c->aligned = (c->P.d % 4 == 0) && aligned16(x) && aligned16(xw) && aligned16(mem) && aligned16(anchors);
    c->bound = true;
    c->compressed = false;
    return QS_OK;
}

int qs_set_sharding(qs_ctx* c, int worker_base, int R_total) {
    if (!c) return QS_INVALID_ARG;
    if (worker_base < 0 || R_total > MAX_R || worker_base + c->P.R > R_total)
        return fail(c, QS_INVALID_ARG, "need 0 <= worker_base and worker_base + R <= R_total <= 32");
    c->P.wbase = worker_base;
    c->P.rdiv = R_total;
    c->compressed = false;
    return QS_OK;
}

int qs_local_step(qs_ctx* c, const float* grad, float eta, const uint8_t* worker_mask) {
    if (!c || !grad) return fail(c, QS_INVALID_ARG, "grad is required");
    if (!c->bound) return fail(c, QS_STATE, "no buffers bound");
    Active act;
    if (!make_active(c, worker_mask, &act)) return QS_OK;
    const StepArgs sa = {grad, nullptr, eta, 0.0f};
    launch_local_step(c->P, act, sa, c->aligned && aligned16(grad), c->sms, c->st);
    return after_launch(c, 1, "local_step");
}

int qs_local_step_momentum(qs_ctx* c, const float* grad, float* vel, float eta, float mu, const uint8_t* worker_mask) {
    if (!c || !grad || !vel) return fail(c, QS_INVALID_ARG, "grad and vel are required");
    if (!c->bound) return fail(c, QS_STATE, "no buffers bound");
    Active act;
    if (!make_active(c, worker_mask, &act)) return QS_OK;
    const StepArgs sa = {grad, vel, eta, mu};
    launch_local_step(c->P, act, sa, c->aligned && aligned16(grad) && aligned16(vel), c->sms, c->st);
    return after_launch(c, 1, "local_step");
}

int qs_compress_feedback(qs_ctx* c, uint64_t round, const uint8_t* worker_mask) {
    if (!c) return QS_INVALID_ARG;
    if (!c->bound) return fail(c, QS_STATE, "no buffers bound");
    if (round != QS_ROUND_AUTO && round >= (1ull << 56)) return fail(c, QS_INVALID_ARG, "round must be below 2^56");
    Active act;
    if (!make_active(c, worker_mask, &act)) { c->last = act; c->compressed = true; return QS_OK; }
    return round_body(c, take_round(c, round), act, false, nullptr, 0, nullptr);
}

int qs_pack(qs_ctx* c, uint32_t* wire, int64_t stride_words, int64_t* bits_out) {
    if (!c || !wire) return fail(c, QS_INVALID_ARG, "wire is required");
    if (!c->compressed) return fail(c, QS_STATE, "nothing compressed yet");
    if (stride_words < c->wire_words) return fail(c, QS_CAPACITY, "stride_words is below qs_wire_words");
    if (c->last.n == 0) return QS_OK;
    return run_mid(c, c->last, 0, 1, 0, 0, wire, stride_words, bits_out);
}

int qs_unpack_accumulate(qs_ctx* c, const uint32_t* wire, int64_t stride_words, const uint8_t* worker_mask) {
    if (!c || !wire) return fail(c, QS_INVALID_ARG, "wire is required");
    if (!c->bound) return fail(c, QS_STATE, "no buffers bound");
    if (stride_words < c->wire_words) return fail(c, QS_CAPACITY, "stride_words is below qs_wire_words");
    Active act;
    if (!make_active_job(c, worker_mask, &act)) return QS_OK;
    return run_mid(c, act, 0, 0, 1, 0, const_cast<uint32_t*>(wire), stride_words, nullptr);
}

int qs_broadcast(qs_ctx* c, const uint8_t* worker_mask) {
    if (!c) return QS_INVALID_ARG;
    if (!c->bound) return fail(c, QS_STATE, "no buffers bound");
    Active act;
    if (!make_active(c, worker_mask, &act)) return QS_OK;
    launch_broadcast(c->P, act, c->aligned, c->sms, c->st);
    return after_launch(c, 1, "broadcast");
}

int qs_sync_round(qs_ctx* c, uint64_t round, const uint8_t* worker_mask, uint32_t* wire, int64_t stride_words,
                  int64_t* bits_out) {
    if (!c || !wire) return fail(c, QS_INVALID_ARG, "wire is required");
    if (!c->bound) return fail(c, QS_STATE, "no buffers bound");
    if (stride_words < c->wire_words) return fail(c, QS_CAPACITY, "stride_words is below qs_wire_words");
    if (round != QS_ROUND_AUTO && round >= (1ull << 56)) return fail(c, QS_INVALID_ARG, "round must be below 2^56");
    if (c->P.rdiv != c->P.R) return fail(c, QS_STATE, "a sharded context runs the separate calls: the records of the other shards are needed");
    Active act;
    if (!make_active(c, worker_mask, &act)) return QS_OK;
    return round_body(c, take_round(c, round), act, true, wire, stride_words, bits_out);
}

int qs_sync_round_step(qs_ctx* c, const float* grad, float* vel, float eta, float mu, uint64_t round,
                       const uint8_t* worker_mask, uint32_t* wire, int64_t stride_words, int64_t* bits_out) {
    if (!c || !wire || !grad) return fail(c, QS_INVALID_ARG, "grad and wire are required");
    if (!c->bound) return fail(c, QS_STATE, "no buffers bound");
    if (stride_words < c->wire_words) return fail(c, QS_CAPACITY, "stride_words is below qs_wire_words");
    if (round != QS_ROUND_AUTO && round >= (1ull << 56)) return fail(c, QS_INVALID_ARG, "round must be below 2^56");
    if (c->P.rdiv != c->P.R) return fail(c, QS_STATE, "a sharded context runs the separate calls: the records of the other shards are needed");
    Active act;
    if (!make_active(c, worker_mask, &act)) return QS_OK;
    const StepArgs sa = {grad, vel, eta, mu};
    return round_body(c, take_round(c, round), act, true, wire, stride_words, bits_out, &sa);
}

int qs_enable_phase_timing(qs_ctx* c, int on) {
    if (!c) return QS_INVALID_ARG;
    fold_timing(c);
    if (on && c->ev.empty()) {
        c->ev.resize((size_t)TIMING_ROUNDS * TIMING_MARKS);
        for (auto& e : c->ev) QS_CUDA_TRY(c, cudaEventCreate(&e));
    }
    c->timing = on != 0;
    return QS_OK;
}

int qs_get_phase_timing(qs_ctx* c, double* ms, int n) {
    if (!c || !ms) return QS_INVALID_ARG;
    fold_timing(c);
    const double v[3] = {c->phase_ms[0], c->phase_ms[1], (double)c->timed_rounds};
    for (int i = 0; i < n && i < 3; ++i) ms[i] = v[i];
    for (double& a : c->phase_ms) a = 0.0;
    c->timed_rounds = 0;
    return QS_OK;
}

int qs_export_selection(qs_ctx* c, int64_t* sel_idx, int32_t* level, uint8_t* sign, float* norm, int64_t* n) {
    if (!c) return QS_INVALID_ARG;
    if (!c->compressed) return fail(c, QS_STATE, "nothing compressed yet");
    launch_export(c->P, (long long*)sel_idx, level, sign, norm, (long long*)n, c->sms, c->st);
    return after_launch(c, 1, "export");
}

int64_t qs_wire_words(const qs_ctx* c) { return c ? c->wire_words : (int64_t)QS_INVALID_ARG; }

int64_t qs_record_bits(const qs_ctx* c, const int64_t* n) {
    if (!c || !n) return QS_INVALID_ARG;
    int64_t bits = 0;
    for (int g = 0; g < c->P.nseg; ++g) {
        const int bi = std::max(1, ceil_log2((uint64_t)(c->off[g + 1] - c->off[g])));
        bits += 64 + n[g] * (int64_t)entry_bits((uint32_t)bi, (uint32_t)c->P.bl, c->P.qz);
    }
    return bits;
}

int64_t qs_gap_words(const qs_ctx* c) { return c ? c->gap_words : (int64_t)QS_INVALID_ARG; }

int qs_recode_gaps(qs_ctx* c, const uint32_t* wire, int64_t stride_words, const uint8_t* worker_mask, uint32_t* packed,
                   int64_t packed_stride, int64_t* bits_out) {
    if (!c || !wire || !packed) return fail(c, QS_INVALID_ARG, "wire and packed are required");
    if (stride_words < c->wire_words) return fail(c, QS_CAPACITY, "stride_words is below qs_wire_words");
    if (packed_stride < c->gap_words) return fail(c, QS_CAPACITY, "packed_stride is below qs_gap_words");
    Active act;
    if (!make_active(c, worker_mask, &act)) return QS_OK;   // the sender's side: this context's workers
    for (int i = 0; i < act.n; ++i)       // words after a record are zero
        QS_CUDA_TRY(c, cudaMemsetAsync(packed + (size_t)act.r[i] * packed_stride, 0, (size_t)c->gap_words * 4, c->st));
    const cudaError_t e = launch_recode_gaps(c->P, act, wire, stride_words, packed, packed_stride,
                                             reinterpret_cast<long long*>(bits_out), c->longest_k, c->most_words, c->row_chunks, c->st);
    if (e != cudaSuccess) return cuda_fail(c, e, "gap-coded records");
    return after_launch(c, 6, "gap-coded records");
}

int qs_decode_gaps(qs_ctx* c, const uint32_t* packed, int64_t packed_stride, const uint8_t* worker_mask, uint32_t* wire,
                   int64_t stride_words) {
    if (!c || !wire || !packed) return fail(c, QS_INVALID_ARG, "wire and packed are required");
    if (stride_words < c->wire_words) return fail(c, QS_CAPACITY, "stride_words is below qs_wire_words");
    if (packed_stride < c->gap_words) return fail(c, QS_CAPACITY, "packed_stride is below qs_gap_words");
    Active act;
    if (!make_active_job(c, worker_mask, &act)) return QS_OK;
    for (int i = 0; i < act.n; ++i)       // the index fields are or-ed into zeroed words
        QS_CUDA_TRY(c, cudaMemsetAsync(wire + (size_t)act.r[i] * stride_words, 0, (size_t)c->wire_words * 4, c->st));
    const cudaError_t e = launch_decode_gaps(c->P, act, packed, packed_stride, wire, stride_words, c->longest_k,
                                             c->most_words, c->row_chunks, c->st);
    if (e != cudaSuccess) return cuda_fail(c, e, "plain records from gap-coded ones");
    return after_launch(c, 6, "plain records from gap-coded ones");
}

int64_t qs_total_k(const qs_ctx* c) { return c ? (int64_t)c->P.K : (int64_t)QS_INVALID_ARG; }

int qs_sync_status(qs_ctx* c) {
    if (!c) return QS_INVALID_ARG;
    QS_CUDA_TRY(c, cudaStreamSynchronize(c->st));
    int code = 0;
    QS_CUDA_TRY(c, cudaMemcpy(&code, c->P.status, sizeof(int), cudaMemcpyDeviceToHost));
    if (code != QS_OK) {
        c->err = code == QS_NONFINITE ? "non-finite value reached the compressor" : "device-side check failed";
        c->compressed = false;
        const int rc = rezero(c);
        if (rc != QS_OK) return rc;
        QS_CUDA_TRY(c, cudaStreamSynchronize(c->st));
    }
    return code;
}

const char* qs_last_error(const qs_ctx* c) { return c ? c->err.c_str() : "null context"; }

uint64_t qs_get_round(const qs_ctx* c) { return c ? c->round : 0; }

int qs_set_round(qs_ctx* c, uint64_t round) {
    if (!c || round >= (1ull << 56)) return QS_INVALID_ARG;
    c->round = round;
    return QS_OK;
}

int qs_get_stage_trace(qs_ctx* c, double* us, int n) {
    if (!c || !us) return QS_INVALID_ARG;
    QS_CUDA_TRY(c, cudaStreamSynchronize(c->st));
    unsigned long long t[TRACE_SLOTS];
    QS_CUDA_TRY(c, cudaMemcpy(t, c->P.trace, sizeof(t), cudaMemcpyDeviceToHost));
    // slot 0 = kernel start, slots 1.. = barriers in order (0 = not reached), last slot = kernel end
    for (int i = 0; i < n && i < TRACE_SLOTS; ++i) us[i] = t[i] ? (double)(t[i] - t[0]) * 1e-3 : -1.0;
    return QS_OK;
}

int qs_get_stats(qs_ctx* c, int64_t* out, int n) {
    if (!c || !out) return QS_INVALID_ARG;
    QS_CUDA_TRY(c, cudaStreamSynchronize(c->st));
    long long dev[2] = {0, 0};
    QS_CUDA_TRY(c, cudaMemcpy(dev, c->P.stats, sizeof(dev), cudaMemcpyDeviceToHost));
    const int64_t v[5] = {c->rounds, (int64_t)dev[0], (int64_t)dev[1], c->launches, (int64_t)c->mid_grid};
    for (int i = 0; i < n && i < 5; ++i) out[i] = v[i];
    return QS_OK;
}

void qs_destroy(qs_ctx* c) {
    if (!c) return;
    cudaStreamSynchronize(c->st);
    for (auto& e : c->ev) cudaEventDestroy(e);
    release(c);
    delete c;
}

}  // extern "C"
