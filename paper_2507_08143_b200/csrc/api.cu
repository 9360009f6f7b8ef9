// Host entry points of the C ABI declared in compactor.h: argument checking, workspace layout
// and kernel sequencing.  No device memory is allocated here.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <vector>

#include "common.cuh"
#include "sm100.cuh"

using namespace compactor;

namespace {

constexpr size_t kAlign = 256;
constexpr int kFallbackSmCount = 148;     // B200, if the device cannot be asked
constexpr int kFusedMaxMp = 48;           // widest padded sketch the fused sweep holds in shared memory
constexpr int kPieceTokens = 1024;        // piece length of the fused sweep, doubled for very long sequences
constexpr int kMaxPiecesPerUnit = 160;
constexpr int kMaxCtas = 256;             // upper bound on the CTAs of the fused sweep (one per SM)
constexpr size_t kL2WindowBytes = (size_t)64 << 20;   // keys that may wait in L2 between their two reads

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Number of SMs of the current device (asked once per device).
int sm_count() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return kFallbackSmCount;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = kFallbackSmCount;
        cached[dev] = n;
    }
    return cached[dev];
}

}  // namespace
namespace compactor {
// COMPACTOR_NO_PDL=1 launches every kernel fully serialised (a measuring aid).
// Chained launches pay where a call's grids do not fill the GPU for long (its kernels are then a chain of
// latencies); on the large workloads they were measured to cost time (C3 +3.5 %, C4 +9 % with every kernel
// chained), so a call chains its kernels only if its keys are at most this many bytes.
constexpr long long kChainMaxKeyBytes = 600LL << 20;
thread_local bool t_chain = false;        // set by make_plan() for the call that this thread is making
bool pdl_enabled(int which) {
    const char* e = getenv("COMPACTOR_NO_PDL");
    if (e != nullptr && e[0] == '1') return false;
    const char* m = getenv("COMPACTOR_PDL_MASK");               // tuning aid: chain these kernels whatever the size
    if (m != nullptr) return (strtol(m, nullptr, 10) & which) != 0;
    return t_chain;
}
void set_chain_for(long long key_bytes) { t_chain = key_bytes <= kChainMaxKeyBytes; }
}  // namespace compactor
namespace {

// Slices per score vector for the selection spread over several CTAs: enough CTAs for two per SM, no
// slice shorter than 8192 scores.
constexpr int kMaxSelectParts = 64;
int select_parts(long long vectors, long long max_n) {
    const long long want = (2LL * sm_count() + vectors - 1) / (vectors > 0 ? vectors : 1);
    long long parts = want < 1 ? 1 : want;
    if (parts > max_n / 8192) parts = max_n / 8192;
    if (parts > kMaxSelectParts) parts = kMaxSelectParts;
    return parts < 1 ? 1 : (int)parts;
}
long long longest_sequence(const compactor_shape* s) {
    long long m = 0;
    for (int b = 0; b < s->batch; ++b) m = std::max<long long>(m, s->cu_seqlens[b + 1] - s->cu_seqlens[b]);
    return m;
}

// The fused persistent sweep is switched on with COMPACTOR_FUSED_SWEEP=1 (it does not yet beat the
// separate kernels; see sweep.cu).
// 0: separate kernels; 1: one launch (Gram, factor and scoring pieces interleaved, keys meant to stay in L2);
// 2: two launches of the same kernel (Gram pieces with the factor tasks hidden behind them, then scoring pieces).
int fused_sweep_mode() {
    const char* e = getenv("COMPACTOR_FUSED_SWEEP");
    if (e == nullptr) return 0;
    return e[0] == '1' ? 1 : (e[0] == '2' ? 2 : 0);
}
bool fused_sweep_enabled() { return fused_sweep_mode() != 0; }

struct HostPlan {
    Plan plan;
    std::vector<int> tables;       // cu_seqlens | cu_keep | cu_chunks | cu_schunks, each batch+1
    size_t off_tables, off_w, off_gpart, off_partials, off_scores, total_bytes;
    int units;
    long long max_n;               // longest sequence
    // fused sweep (Cholesky route, padded sketch of at most kFusedMaxMp columns)
    bool fused;
    int slices, window, n_slots, max_pieces, resident16;
    long long total_pieces;
    size_t off_sched, sched_bytes, off_tbuf;
};

// Workspace layout of the fused sweep for the plan's current window.
void layout_fused(HostPlan* hp) {
    const Plan& p = hp->plan;
    const int nb1 = p.batch + 1;
    // claims may run past the window by one piece per CTA
    const long long want = (long long)hp->window + kMaxCtas;
    const long long slots = hp->total_pieces < want ? hp->total_pieces : want;
    hp->n_slots = (int)(slots < 1 ? 1 : slots);
    size_t off = 0;
    hp->off_tables = off;   off += align_up(sizeof(int) * 4 * nb1);
    hp->off_sched = off;    hp->sched_bytes = sizeof(SweepSched) + sizeof(int) * 5 * (size_t)hp->units;
                            off += align_up(hp->sched_bytes);
    hp->off_w = off;        off += align_up(sizeof(__nv_bfloat16) * w_elems_per_unit(p.mp) * hp->units);
    hp->off_tbuf = off;     off += align_up(sizeof(double) * kD * p.mp * (size_t)hp->units);
    hp->off_partials = off; off += align_up(sizeof(float) * kGramElems * (size_t)hp->n_slots);
    hp->off_gpart = hp->off_partials;
    hp->off_scores = off;   off += align_up(sizeof(float) * (size_t)p.total_tokens * p.layers * p.heads);
    hp->total_bytes = off;
}

bool shape_ok(const compactor_shape* s, int* err) {
    if (s == nullptr || s->cu_seqlens == nullptr) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    if (s->layers < 1 || s->heads < 1 || s->batch < 1) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    if ((long long)s->layers * s->heads > 65535) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    if (s->d != kD || s->m < 1 || s->m > kMaxM) { *err = COMPACTOR_E_UNSUPPORTED; return false; }
    if (s->cu_seqlens[0] != 0) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    for (int b = 0; b < s->batch; ++b)
        if (s->cu_seqlens[b + 1] < s->cu_seqlens[b]) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    if ((long long)s->layers * s->heads * s->batch > 0x7fffffffLL) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    return true;
}

// Fills everything that depends on the shape alone (keep counts are added by the caller).
// `allow_fused`: lay the workspace out for the fused sweep when the sketch is narrow enough.
bool make_plan(const compactor_shape* s, HostPlan* hp, int* err, bool allow_fused = true) {
    if (!shape_ok(s, err)) return false;
    Plan& p = hp->plan;
    memset(&p, 0, sizeof(p));
    p.layers = s->layers; p.heads = s->heads; p.batch = s->batch;
    p.m = s->m; p.mp = s->m <= 64 ? (s->m + 15) / 16 * 16 : 128;
    p.total_tokens = s->cu_seqlens[s->batch];
    hp->max_n = longest_sequence(s);
    compactor::set_chain_for((long long)s->layers * s->heads * p.total_tokens * kD * 2);
    hp->units = s->layers * s->heads * s->batch;
    hp->fused = allow_fused && p.mp <= kFusedMaxMp && fused_sweep_enabled();
    // the one-kernel sweep has no pivoted factorisation and no fp64 scores for sequences about as short as the sketch is
    // wide: a batch with one of those takes the separate kernels
    for (int b = 0; b < s->batch && hp->fused; ++b) {
        const int n = s->cu_seqlens[b + 1] - s->cu_seqlens[b];
        if (n > 0 && n <= s->m + kTinyExtra) hp->fused = false;
    }
    hp->slices = 0; hp->window = 0; hp->n_slots = 0; hp->max_pieces = 0; hp->total_pieces = 0;
    hp->off_sched = 0; hp->sched_bytes = 0; hp->off_tbuf = 0;

    if (hp->fused) {
        // Pieces of 1024 tokens keep the keys that wait between their two reads within L2; sequences beyond
        // 160 pieces get longer ones (their keys outlive L2 anyway) so that the ring of partials stays small.
        long long n_max = 0;
        for (int b = 0; b < s->batch; ++b) {
            const long long n = s->cu_seqlens[b + 1] - s->cu_seqlens[b];
            if (n > n_max) n_max = n;
        }
        int piece = kPieceTokens;
        if (const char* e = getenv("COMPACTOR_PIECE_TOKENS")) {         // tuning aid: 1024, 2048, 4096, ...
            const long v = strtol(e, nullptr, 10);
            if (v >= kPieceTokens && v <= kMaxChunk && (v & (v - 1)) == 0) piece = (int)v;
        }
        while ((n_max + piece - 1) / piece > kMaxPiecesPerUnit && piece < kMaxChunk) piece *= 2;
        const int nb1 = s->batch + 1;
        hp->tables.assign((size_t)4 * nb1, 0);
        int* cs = hp->tables.data();
        int* cc = cs + 2 * nb1;
        long long tc = 0;
        for (int b = 0; b <= s->batch; ++b) cs[b] = s->cu_seqlens[b];
        for (int b = 0; b < s->batch; ++b) {
            tc += (cs[b + 1] - cs[b] + piece - 1) / piece;
            if (tc > 0x7fffffffLL) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
            cc[b + 1] = (int)tc;
        }
        // row slices of a unit's projection: more of them the more partials there are to add up
        int* csl = cs + 3 * nb1;
        for (int b = 0; b < s->batch; ++b) {
            const int pieces = cc[b + 1] - cc[b];
            const int sl = pieces >= 96 ? 32 : pieces >= 48 ? 16 : pieces >= 24 ? 8 : pieces >= 12 ? 4 : pieces >= 4 ? 2 : 1;
            csl[b + 1] = csl[b] + sl;
        }
        hp->total_pieces = tc * s->layers * s->heads;
        if (hp->total_pieces > 0x7fffffffLL) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
        p.chunk = p.schunk = piece;
        p.total_chunks = (int)tc;
        p.total_schunks = csl[s->batch];
        hp->max_pieces = (int)((n_max + piece - 1) / piece);
        hp->slices = p.total_schunks;
        size_t window_bytes = kL2WindowBytes;
        if (const char* e = getenv("COMPACTOR_L2_WINDOW_MIB")) {        // tuning aid
            const long v = strtol(e, nullptr, 10);
            if (v > 0 && v < 65536) window_bytes = (size_t)v << 20;
        }
        hp->resident16 = 16;
        if (const char* e = getenv("COMPACTOR_RESIDENT_16THS")) {       // tuning aid
            const long v = strtol(e, nullptr, 10);
            if (v >= 1 && v <= 16) hp->resident16 = (int)v;
        }
        // the window counts all pieces; only resident16 / 16 of them occupy L2 while they wait
        long long budget = (long long)(window_bytes / ((size_t)piece * kD * sizeof(__nv_bfloat16))) * 16 / hp->resident16;
        if (fused_sweep_mode() == 2) budget = 1024;          // nothing waits in L2: the window only bounds the ring of partial sums
        hp->window = (int)(budget > hp->max_pieces + 1 ? budget : hp->max_pieces + 1);
        layout_fused(hp);
        return true;
    }

    // Block length (tokens per CTA of the two sweeps, one fp64 Gram partial per block): the power
    // of two times 256 that minimises a small cost model - waves of CTAs over the SMs, a fixed
    // set-up cost per CTA, the block's bytes at one SM's share of the bandwidth, and the traffic of
    // the 128 KiB partial that every block writes and the projection reads back.
    auto count_chunks = [&](int c) {
        long long t = 0;
        for (int b = 0; b < s->batch; ++b) {
            long long n = s->cu_seqlens[b + 1] - s->cu_seqlens[b];
            t += (n + c - 1) / c;
        }
        return t;
    };
    // Sequences of one length give CTAs of one duration, which run in waves; a ragged batch gives CTAs of
    // all durations, and then the sweep takes the average load of an SM plus about half a block at its end.
    bool ragged = false;
    for (int b = 1; b < s->batch; ++b)
        ragged = ragged || (s->cu_seqlens[b + 1] - s->cu_seqlens[b]) != (s->cu_seqlens[1] - s->cu_seqlens[0]);
    const double lh = (double)s->layers * s->heads;
    const double stream_us = lh * (double)p.total_tokens * 256.0 / 44e3 / kFallbackSmCount;   // 44 GB/s = 44e3 B/us per SM
    auto ragged_cost = [&](int c, double setup_us) {
        const double ctas = (double)count_chunks(c) * lh;
        const double longest = (double)(hp->max_n < c ? hp->max_n : c);
        return ctas * setup_us / kFallbackSmCount + stream_us + 0.5 * (setup_us + longest * 256.0 / 44e3);
    };
    int chunk = kMaxChunk;
    double best = 1e300;
    for (int c = kMinChunk; c <= kMaxChunk; c *= 2) {
        const double ctas = (double)count_chunks(c) * lh;
        const double waves = ceil(ctas / kFallbackSmCount);
        const double per_cta_us = 4.0 + (double)(hp->max_n < c ? hp->max_n : c) * 256.0 / 44e3;   // a block is never longer than the sequence
        const double partial_us = ctas * 2.0 * 131072.0 / 6.4e6;      // written once, read once (a whole 128 x 128 fp64 matrix at 6.4 TB/s fits the measurements; ten of its sixteen blocks move)
        const double cost = (ragged ? ragged_cost(c, 4.0) : waves * per_cta_us) + partial_us;
        if (cost < best * 0.999) { best = cost; chunk = c; }
    }
    if (const char* e = getenv("COMPACTOR_GRAM_BLOCK")) {               // tuning aid
        const long v = strtol(e, nullptr, 10);
        if (v >= kMinChunk && v <= kMaxChunk && (v & (v - 1)) == 0) chunk = (int)v;
    }
    p.chunk = chunk;
    long long tc = count_chunks(chunk);
    if (tc > 0x7fffffffLL) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    p.total_chunks = (int)tc;
    // The scoring sweep writes no partial sums and sets up faster; its blocks are chosen for balance: the
    // hardware hands out CTAs as SMs free up, so the sweep ends about half a block after the average SM.
    int schunk = kMaxChunk;
    best = 1e300;
    for (int c = kMinChunk; c <= kMaxChunk; c *= 2) {
        const double ctas = (double)count_chunks(c) * lh;
        const double block_bytes = (double)(hp->max_n < c ? hp->max_n : c) * 256.0;
        const double per_cta_us = 2.0 + block_bytes / 44e3;
        double cost = ragged ? ragged_cost(c, 2.0)
                             : (ctas / kFallbackSmCount < 1.0 ? 1.0 : ctas / kFallbackSmCount) * per_cta_us + 0.5 * per_cta_us;
        if (!ragged && ctas <= 2.0 * kFallbackSmCount) {
            // Two CTAs of this sweep fit on an SM, so these are all resident at once and nothing runs in waves: every
            // SM streams its q or q + 1 blocks at its share of the bandwidth, one SM alone at 60 GB/s at most (measured:
            // 112 CTAs of 8 MB reach 6.3 TB/s; 224 take as long as this says).
            const double sms = kFallbackSmCount, cap = 60e3, all = 6.4e6;
            const double q = floor(ctas / sms), more = ctas - q * sms;            // `more` SMs have q + 1 blocks
            const double t1 = q * block_bytes / (all / sms < cap ? all / sms : cap);       // until the SMs with q blocks are done
            const double t2 = more > 0 ? block_bytes / (all / more < cap ? all / more : cap) : 0.0;
            cost = 2.0 + t1 + t2;
        }
        if (cost < best * 0.999) { best = cost; schunk = c; }
    }
    if (const char* e = getenv("COMPACTOR_SCORE_BLOCK")) {              // tuning aid
        const long v = strtol(e, nullptr, 10);
        if (v >= kMinChunk && v <= kMaxChunk && (v & (v - 1)) == 0) schunk = (int)v;
    }
    p.schunk = schunk;
    tc = count_chunks(schunk);
    if (tc > 0x7fffffffLL) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    p.total_schunks = (int)tc;

    const int nb1 = s->batch + 1;
    hp->tables.assign((size_t)4 * nb1, 0);
    int* cs = hp->tables.data();
    int* cc = cs + 2 * nb1;
    int* csc = cs + 3 * nb1;
    for (int b = 0; b <= s->batch; ++b) cs[b] = s->cu_seqlens[b];
    for (int b = 0; b < s->batch; ++b) cc[b + 1] = cc[b] + (cs[b + 1] - cs[b] + chunk - 1) / chunk;
    for (int b = 0; b < s->batch; ++b) csc[b + 1] = csc[b] + (cs[b + 1] - cs[b] + schunk - 1) / schunk;

    size_t off = 0;
    hp->off_tables = off;   off += align_up(sizeof(int) * 4 * nb1);
    hp->off_w = off;        off += align_up(sizeof(__nv_bfloat16) * w_elems_per_unit(p.mp) * hp->units);
    hp->off_gpart = off;    off += align_up(sizeof(double) * a_elems_per_unit(p.mp) * hp->units);   // the parts of A = Phi^T M Phi per unit
    hp->off_partials = off; off += align_up(sizeof(double) * kGramElems * (size_t)p.total_chunks * s->layers * s->heads);
    hp->off_scores = off;   off += align_up(sizeof(float) * (size_t)p.total_tokens * s->layers * s->heads);
    hp->total_bytes = off;
    return true;
}

bool set_keep(const compactor_shape* s, const int32_t* keep, HostPlan* hp) {
    if (keep == nullptr) return false;
    const int nb1 = s->batch + 1;
    int* ck = hp->tables.data() + nb1;
    long long tot = 0;
    for (int b = 0; b < s->batch; ++b) {
        int n = s->cu_seqlens[b + 1] - s->cu_seqlens[b];
        if (keep[b] < 0 || keep[b] > n) return false;
        tot += keep[b];
        ck[b + 1] = (int)tot;
    }
    hp->plan.total_keep = (int)tot;
    return true;
}

bool mat_ok(const compactor_mat& m) {
    if (m.ptr == nullptr || ((uintptr_t)m.ptr & 15) != 0) return false;
    if (m.stride_token < kD || (m.stride_token & 7) || (m.stride_layer & 7) || (m.stride_head & 7)) return false;
    if (m.stride_layer < 0 || m.stride_head < 0) return false;
    return true;
}

Mat to_mat(const compactor_mat& m) {
    Mat r;
    r.ptr = static_cast<const __nv_bfloat16*>(m.ptr);
    r.stride_layer = m.stride_layer; r.stride_head = m.stride_head; r.stride_token = m.stride_token;
    return r;
}

// The tables travel to the device as kernel arguments, kInlineTableInts entries per launch: no copy from
// host memory is enqueued, so the call never makes the runtime wait for the stream and can be recorded
// into a CUDA graph and replayed, whatever the batch size.
constexpr int kInlineTableInts = 960;
struct InlineTables { int n; int v[kInlineTableInts]; };
__global__ void write_tables_kernel(const __grid_constant__ InlineTables t, int* __restrict__ dst) {
    for (int i = threadIdx.x; i < t.n; i += blockDim.x) dst[i] = t.v[i];
}

// Puts the tables at the head of the workspace and points the plan at them.
cudaError_t upload_tables(HostPlan* hp, void* ws, cudaStream_t stream) {
    const int nb1 = hp->plan.batch + 1;
    int* dev = reinterpret_cast<int*>(static_cast<char*>(ws) + hp->off_tables);
    const long long total = 4LL * nb1;
    for (long long done = 0; done < total; done += kInlineTableInts) {
        InlineTables t;
        t.n = (int)(total - done < kInlineTableInts ? total - done : kInlineTableInts);
        memcpy(t.v, hp->tables.data() + done, sizeof(int) * t.n);
        write_tables_kernel<<<1, 256, 0, stream>>>(t, dev + done);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    hp->plan.cu_seqlens = dev;
    hp->plan.cu_keep = dev + nb1;
    hp->plan.cu_chunks = dev + 2 * nb1;
    hp->plan.cu_schunks = dev + 3 * nb1;
    return cudaSuccess;
}

#define CK(expr) do { cudaError_t e__ = (expr); if (e__ != cudaSuccess) return COMPACTOR_E_CUDA; } while (0)

// Optional stage markers: caller-created events recorded on the stream between kernels.
struct Marks {
    void* const* ev = nullptr;
    int n = 0;
    cudaError_t mark(int i, cudaStream_t st) const {
        if (ev == nullptr || i >= n || ev[i] == nullptr) return cudaSuccess;
        return cudaEventRecord(static_cast<cudaEvent_t>(ev[i]), st);
    }
};

#ifdef COMPACTOR_SWEEP_PROFILE
long long* g_sweep_profile = nullptr;     // instrumented builds only: per-CTA cycle counters
#endif

int run_scoring(HostPlan& hp, const Mat& k, const float* phi, const float* attn, float lambda,
                float* scores, int32_t* status, char* ws, cudaStream_t stream, const Marks& mk = Marks(),
                int factorization = COMPACTOR_FACTOR_CHOLESKY, double eig_floor = 0.0, bool clear_status = true) {
    __nv_bfloat16* w = reinterpret_cast<__nv_bfloat16*>(ws + hp.off_w);
    if (status != nullptr && clear_status) CK(cudaMemsetAsync(status, 0, sizeof(int32_t) * hp.units, stream));
    if (hp.fused) {
        // one persistent kernel: Gram pieces, factorisation and scoring pieces from a common work queue
        if (factorization != COMPACTOR_FACTOR_CHOLESKY) return COMPACTOR_E_INVALID_ARGUMENT;
        CK(cudaMemsetAsync(ws + hp.off_sched, 0, hp.sched_bytes, stream));
        SweepArgs a;
        memset(&a, 0, sizeof(a));
        a.p = hp.plan; a.k = k;
        a.units = hp.units; a.total_pieces = (int)hp.total_pieces;
        a.total_ftasks = hp.plan.total_schunks * hp.plan.layers * hp.plan.heads;
        a.window = hp.window; a.n_slots = hp.n_slots; a.resident16 = hp.resident16;
        a.sched = reinterpret_cast<SweepSched*>(ws + hp.off_sched);
        a.gram_done = reinterpret_cast<int*>(ws + hp.off_sched + sizeof(SweepSched));
        a.slices_claimed = a.gram_done + hp.units;
        a.slices_done = a.slices_claimed + hp.units;
        a.score_claimed = a.slices_done + hp.units;
        a.w_ready = a.score_claimed + hp.units;
        a.partials = reinterpret_cast<float*>(ws + hp.off_partials);
        a.t_buf = reinterpret_cast<double*>(ws + hp.off_tbuf);
        a.w = w; a.phi = phi; a.scores = scores; a.status = status;
#ifdef COMPACTOR_SWEEP_PROFILE
        a.prof = g_sweep_profile;
#endif
        const int ctas = sm_count() < kMaxCtas ? sm_count() : kMaxCtas;
        CK(mk.mark(0, stream));
        if (fused_sweep_mode() == 2) {
            a.phase = 1;
            CK(launch_sweep(a, ctas, stream));
            CK(mk.mark(1, stream));             // Gram pieces with the factor tasks behind them
            CK(mk.mark(2, stream));
            a.phase = 2;
            CK(launch_sweep(a, ctas, stream));
            CK(mk.mark(3, stream));
        } else {
            a.phase = 0;
            CK(launch_sweep(a, ctas, stream));
            CK(mk.mark(1, stream));             // the one kernel does all three steps: the whole time shows as the first
            CK(mk.mark(2, stream));
            CK(mk.mark(3, stream));
        }
    } else {
        double* partials = reinterpret_cast<double*>(ws + hp.off_partials);
        CK(mk.mark(0, stream));
        CK(launch_gram(hp.plan, k, partials, status, stream));
        CK(mk.mark(1, stream));
        CK(launch_factor(hp.plan, k, partials, phi, reinterpret_cast<double*>(ws + hp.off_gpart), w, scores, status,
                         factorization, eig_floor, sm_count(), stream));
        CK(mk.mark(2, stream));
        CK(launch_score(hp.plan, k, w, scores, status, factorization == COMPACTOR_FACTOR_CHOLESKY, stream));
        CK(mk.mark(3, stream));
    }
    if (attn != nullptr) {
        // a few long units: cut into slices (W and the Gram partials are dead by now; their place holds the slices' statistics)
        int parts = 1;
        if (2 * hp.units <= sm_count() && hp.max_n >= 65536) parts = select_parts(hp.units, hp.max_n);
        if (sizeof(double) * 4 * (size_t)hp.units * parts > hp.off_scores - hp.off_w) parts = 1;
        CK(launch_blend(hp.plan, attn, lambda, scores, parts, reinterpret_cast<double*>(ws + hp.off_w), stream));
    }
    CK(mk.mark(4, stream));
    return COMPACTOR_OK;
}

// Per-head selection.  One CTA per unit keeps every SM busy when there are many units; a few long
// units (one layer of a long context) are cut into slices instead, which needs `scratch` for the shared
// histograms and candidate lists.  Both routes give the same indices.
cudaError_t select_per_head(const HostPlan& hp, const compactor_shape* shape, const float* scores, int* idx,
                            char* scratch, size_t scratch_bytes, cudaStream_t st) {
    // rough costs in microseconds: one CTA walks a unit's scores four times; the sliced route pays four small launches
    // and then shares all scores between the SMs
    const long long max_n = longest_sequence(shape);
    const double t_single = 12.0 + 0.37e-3 * (double)max_n;
    const double t_sliced = 40.0 + 6.0e-6 * (double)hp.plan.total_tokens * shape->layers * shape->heads;
    if (hp.units <= sm_count() && t_sliced < 0.8 * t_single && scratch != nullptr) {
        const int parts = select_parts(hp.units, max_n);
        const MultiSelectLayout l = multi_select_layout(shape->layers, shape->heads, shape->batch, hp.plan.total_tokens,
                                                        false, kMaxSelectParts);
        if (parts > 1 && l.total <= scratch_bytes)
            return launch_select_multi(hp.plan, scores, idx, nullptr, multi_select_at(scratch, l, parts, false), st);
    }
    return launch_select(hp.plan, scores, idx, st);
}

// Selection across heads: always the route with one CTA per (head, slice).
cudaError_t select_across(const HostPlan& hp, const compactor_shape* shape, const float* scores, int* idx,
                          int* head_offsets, char* scratch, cudaStream_t st) {
    const int parts = select_parts(hp.units, longest_sequence(shape));
    const MultiSelectLayout l = multi_select_layout(shape->layers, shape->heads, shape->batch, hp.plan.total_tokens,
                                                    true, kMaxSelectParts);
    return launch_select_multi(hp.plan, scores, idx, head_offsets, multi_select_at(scratch, l, parts, true), st);
}
size_t across_scratch_bytes(const compactor_shape* shape, long long total_tokens) {
    return multi_select_layout(shape->layers, shape->heads, shape->batch, total_tokens, true, kMaxSelectParts).total;
}

}  // namespace

#ifdef COMPACTOR_SWEEP_PROFILE
extern "C" void compactor_debug_set_profile_buffer(long long* device_counters) { g_sweep_profile = device_counters; }
#endif

extern "C" {

int compactor_version(void) { return 100; }

const char* compactor_error_string(int code) {
    switch (code) {
        case COMPACTOR_OK: return "ok";
        case COMPACTOR_E_INVALID_ARGUMENT: return "invalid argument";
        case COMPACTOR_E_UNSUPPORTED: return "unsupported shape (d must be 128, 1 <= m <= 128)";
        case COMPACTOR_E_WORKSPACE: return "workspace too small";
        case COMPACTOR_E_CUDA: return "CUDA runtime error";
        case COMPACTOR_E_TOO_LARGE: return "problem needs more scratch than the built-in 32 MiB array holds";
        default: return "unknown status";
    }
}

int compactor_make_sketch(uint64_t seed, int32_t d, int32_t m, float* phi_host) {
    if (phi_host == nullptr || d < 1 || m < 1) return COMPACTOR_E_INVALID_ARGUMENT;
    auto word = [seed](uint64_t i) {
        uint64_t z = seed + (i + 1) * 0x9E3779B97F4A7C15ull;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        return z ^ (z >> 31);
    };
    const long long count = (long long)d * m;
    const double root_m = sqrt((double)m);
    const double two_pi = 6.283185307179586476925286766559;
    for (long long pidx = 0; 2 * pidx < count; ++pidx) {
        double u1 = (double)((word(2 * pidx) >> 11) + 1) * 0x1.0p-53;
        double u2 = (double)(word(2 * pidx + 1) >> 11) * 0x1.0p-53;
        double rad = sqrt(-2.0 * log(u1));
        phi_host[2 * pidx] = (float)(rad * cos(two_pi * u2) / root_m);
        if (2 * pidx + 1 < count) phi_host[2 * pidx + 1] = (float)(rad * sin(two_pi * u2) / root_m);
    }
    return COMPACTOR_OK;
}

int64_t compactor_keep_count(int64_t n, double r) {
    if (n <= 0) return 0;
    double c = ceil(r * (double)n);
    if (!(c >= 1.0)) return 1;          // also catches NaN
    if (c >= (double)n) return n;
    return (int64_t)c;
}

int compactor_calibrated_ratio(double nll, double alpha, double beta, double tau, double* r_out) {
    if (r_out == nullptr || !(tau > 0.0) || !(tau <= 1.0)) return COMPACTOR_E_INVALID_ARGUMENT;
    const double b = alpha * nll + beta;
    if (!isfinite(b)) return COMPACTOR_E_INVALID_ARGUMENT;
    *r_out = (b == 0.0) ? tau : log1p(tau * expm1(b)) / b;
    return COMPACTOR_OK;
}

size_t compactor_workspace_bytes(const compactor_shape* shape) {
    // enough for either route: the fused sweep and the separate kernels of the variants
    HostPlan hp; int err = 0;
    if (!make_plan(shape, &hp, &err, false)) return 0;
    const size_t separate = hp.total_bytes;
    if (!make_plan(shape, &hp, &err, true)) return 0;
    return hp.total_bytes > separate ? hp.total_bytes : separate;
}

int compactor_score(const compactor_shape* shape, compactor_mat k_score, const float* phi,
                    const float* attn_scores, float lambda, float* scores_out,
                    int32_t* status, void* workspace, size_t workspace_bytes, void* stream) {
    HostPlan hp; int err = 0;
    if (!make_plan(shape, &hp, &err)) return err;
    if (!mat_ok(k_score) || phi == nullptr || scores_out == nullptr || workspace == nullptr)
        return COMPACTOR_E_INVALID_ARGUMENT;
    if (((uintptr_t)workspace & 255) != 0) return COMPACTOR_E_INVALID_ARGUMENT;
    if (workspace_bytes < hp.total_bytes) return COMPACTOR_E_WORKSPACE;
    if (hp.plan.total_tokens == 0) return COMPACTOR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CK(upload_tables(&hp, workspace, st));
    return run_scoring(hp, to_mat(k_score), phi, attn_scores, lambda, scores_out, status,
                       static_cast<char*>(workspace), st);
}

int compactor_score_variant(const compactor_shape* shape, compactor_mat k_score, const float* phi,
                            int32_t factorization, double eig_floor, const float* attn_scores, float lambda,
                            float* scores_out, int32_t* status, void* workspace, size_t workspace_bytes,
                            void* stream) {
    if (factorization == COMPACTOR_FACTOR_CHOLESKY)
        return compactor_score(shape, k_score, phi, attn_scores, lambda, scores_out, status, workspace,
                               workspace_bytes, stream);
    if (factorization != COMPACTOR_FACTOR_EIG) return COMPACTOR_E_INVALID_ARGUMENT;
    if (!(eig_floor > 0.0) || !std::isfinite(eig_floor)) return COMPACTOR_E_INVALID_ARGUMENT;
    HostPlan hp; int err = 0;
    if (!make_plan(shape, &hp, &err, false)) return err;
    if (hp.plan.mp > 64) return COMPACTOR_E_UNSUPPORTED;
    if (!mat_ok(k_score) || phi == nullptr || scores_out == nullptr || workspace == nullptr)
        return COMPACTOR_E_INVALID_ARGUMENT;
    if (((uintptr_t)workspace & 255) != 0) return COMPACTOR_E_INVALID_ARGUMENT;
    if (workspace_bytes < hp.total_bytes) return COMPACTOR_E_WORKSPACE;
    if (hp.plan.total_tokens == 0) return COMPACTOR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CK(upload_tables(&hp, workspace, st));
    return run_scoring(hp, to_mat(k_score), phi, attn_scores, lambda, scores_out, status,
                       static_cast<char*>(workspace), st, Marks(), factorization, eig_floor);
}

int compactor_select(const compactor_shape* shape, const float* scores, const int32_t* keep_counts,
                     int32_t* idx_out, int32_t* status, void* workspace, size_t workspace_bytes, void* stream) {
    (void)status;
    HostPlan hp; int err = 0;
    if (!make_plan(shape, &hp, &err)) return err;
    if (scores == nullptr || idx_out == nullptr || workspace == nullptr || !set_keep(shape, keep_counts, &hp))
        return COMPACTOR_E_INVALID_ARGUMENT;
    if (((uintptr_t)workspace & 255) != 0) return COMPACTOR_E_INVALID_ARGUMENT;
    if (workspace_bytes < hp.off_w) return COMPACTOR_E_WORKSPACE;      // the tables; the rest, if any, is scratch
    if (hp.plan.total_keep == 0) return COMPACTOR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CK(upload_tables(&hp, workspace, st));
    CK(select_per_head(hp, shape, scores, idx_out, static_cast<char*>(workspace) + hp.off_w, workspace_bytes - hp.off_w, st));
    return COMPACTOR_OK;
}

int compactor_compact(const compactor_shape* shape, compactor_mat k_cache, compactor_mat v_cache,
                      const int32_t* idx, const int32_t* keep_counts, void* k_out, void* v_out,
                      void* workspace, size_t workspace_bytes, void* stream) {
    HostPlan hp; int err = 0;
    if (!make_plan(shape, &hp, &err)) return err;
    if (!mat_ok(k_cache) || !mat_ok(v_cache) || idx == nullptr || k_out == nullptr || v_out == nullptr ||
        workspace == nullptr || !set_keep(shape, keep_counts, &hp))
        return COMPACTOR_E_INVALID_ARGUMENT;
    if ((((uintptr_t)k_out | (uintptr_t)v_out) & 15) != 0 || ((uintptr_t)workspace & 255) != 0)
        return COMPACTOR_E_INVALID_ARGUMENT;
    if (workspace_bytes < hp.off_w) return COMPACTOR_E_WORKSPACE;      // only the tables are used
    if (hp.plan.total_keep == 0) return COMPACTOR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CK(upload_tables(&hp, workspace, st));
    CK(launch_compact(hp.plan, to_mat(k_cache), to_mat(v_cache), idx,
                      static_cast<__nv_bfloat16*>(k_out), static_cast<__nv_bfloat16*>(v_out), st));
    return COMPACTOR_OK;
}

static int compress_impl(const compactor_shape* shape, compactor_mat k_score, compactor_mat k_cache,
                         compactor_mat v_cache, const float* phi, const float* attn_scores,
                         float lambda, const int32_t* keep_counts,
                         float* scores_out, int32_t* idx_out, void* k_out, void* v_out,
                         int32_t* status, void* workspace, size_t workspace_bytes, void* stream, const Marks& mk) {
    HostPlan hp; int err = 0;
    if (!make_plan(shape, &hp, &err)) return err;
    if (!mat_ok(k_score) || !mat_ok(k_cache) || !mat_ok(v_cache) || phi == nullptr || idx_out == nullptr ||
        k_out == nullptr || v_out == nullptr || workspace == nullptr || !set_keep(shape, keep_counts, &hp))
        return COMPACTOR_E_INVALID_ARGUMENT;
    if ((((uintptr_t)k_out | (uintptr_t)v_out) & 15) != 0 || ((uintptr_t)workspace & 255) != 0)
        return COMPACTOR_E_INVALID_ARGUMENT;
    if (workspace_bytes < hp.total_bytes) return COMPACTOR_E_WORKSPACE;
    if (hp.plan.total_tokens == 0) return COMPACTOR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    float* scores = scores_out != nullptr ? scores_out : reinterpret_cast<float*>(ws + hp.off_scores);
    CK(upload_tables(&hp, workspace, st));
    int rc = run_scoring(hp, to_mat(k_score), phi, attn_scores, lambda, scores, status, ws, st, mk);
    if (rc != COMPACTOR_OK) return rc;
    // W, the projections and the Gram partials are dead once the scores exist: the selection may use their place
    if (hp.plan.total_keep > 0)
        CK(select_per_head(hp, shape, scores, idx_out, ws + hp.off_w, hp.off_scores - hp.off_w, st));
    CK(mk.mark(5, st));
    if (hp.plan.total_keep > 0)
        CK(launch_compact(hp.plan, to_mat(k_cache), to_mat(v_cache), idx_out,
                          static_cast<__nv_bfloat16*>(k_out), static_cast<__nv_bfloat16*>(v_out), st));
    CK(mk.mark(6, st));
    return COMPACTOR_OK;
}

int compactor_compress(const compactor_shape* shape, compactor_mat k_score, compactor_mat k_cache,
                       compactor_mat v_cache, const float* phi, const float* attn_scores,
                       float lambda, const int32_t* keep_counts,
                       float* scores_out, int32_t* idx_out, void* k_out, void* v_out,
                       int32_t* status, void* workspace, size_t workspace_bytes, void* stream) {
    return compress_impl(shape, k_score, k_cache, v_cache, phi, attn_scores, lambda, keep_counts, scores_out,
                         idx_out, k_out, v_out, status, workspace, workspace_bytes, stream, Marks());
}

int compactor_compress_profiled(const compactor_shape* shape, compactor_mat k_score, compactor_mat k_cache,
                                compactor_mat v_cache, const float* phi, const float* attn_scores,
                                float lambda, const int32_t* keep_counts,
                                float* scores_out, int32_t* idx_out, void* k_out, void* v_out,
                                int32_t* status, void* workspace, size_t workspace_bytes, void* stream,
                                void* const* stage_events, int32_t n_events) {
    if (stage_events == nullptr || n_events < 0) return COMPACTOR_E_INVALID_ARGUMENT;
    Marks mk; mk.ev = stage_events; mk.n = n_events;
    return compress_impl(shape, k_score, k_cache, v_cache, phi, attn_scores, lambda, keep_counts, scores_out,
                         idx_out, k_out, v_out, status, workspace, workspace_bytes, stream, mk);
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Scoring without a caller-provided workspace.
//
// Some hosts of this library may not allocate device memory when they need scores: a serving
// engine that has handed the whole device to its own paged-cache allocator, a plugin running
// under an allocator lock, or code between the begin and end of a stream capture, where
// cudaMalloc is not permitted.  For them the scratch that compactor_score normally takes from
// the caller lives in this fixed array, which every process that loads the library holds on
// each device it uses, until exit.
namespace {

constexpr size_t kBuiltinScratchBytes = (size_t)32 << 20;     // 32 MiB
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];

constexpr int kMaxDevices = 64;
void* g_builtin_scratch_ptr[kMaxDevices] = {};
std::mutex g_builtin_scratch_mutex;

// Device address of the array on the current device.  In host code the array's name is only a
// handle for the runtime, never an address a kernel may use; the real address is asked for once
// per device and remembered.
int builtin_scratch(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return COMPACTOR_E_CUDA;
    std::lock_guard<std::mutex> lock(g_builtin_scratch_mutex);
    if (g_builtin_scratch_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_builtin_scratch) != cudaSuccess || ptr == nullptr) return COMPACTOR_E_CUDA;
        g_builtin_scratch_ptr[dev] = ptr;
    }
    *out = g_builtin_scratch_ptr[dev];
    return COMPACTOR_OK;
}

// Re-derives the chunk-dependent part of a plan for a given Gram block length.
void replan_chunk(const compactor_shape* s, HostPlan* hp, int chunk) {
    Plan& p = hp->plan;
    const int nb1 = s->batch + 1;
    int* cs = hp->tables.data();
    int* cc = cs + 2 * nb1;
    cc[0] = 0;
    for (int b = 0; b < s->batch; ++b) cc[b + 1] = cc[b] + (cs[b + 1] - cs[b] + chunk - 1) / chunk;
    p.chunk = chunk;
    p.total_chunks = cc[s->batch];
    hp->off_scores = hp->off_partials +
                     align_up(sizeof(double) * kGramElems * (size_t)p.total_chunks * s->layers * s->heads);
    hp->total_bytes = hp->off_scores + align_up(sizeof(float) * (size_t)p.total_tokens * s->layers * s->heads);
}

}  // namespace

extern "C" {

size_t compactor_builtin_scratch_bytes(void) { return kBuiltinScratchBytes; }

int compactor_score_builtin_scratch(const compactor_shape* shape, compactor_mat k_score, const float* phi,
                                    const float* attn_scores, float lambda, float* scores_out,
                                    int32_t* status, void* stream) {
    HostPlan hp; int err = 0;
    if (!make_plan(shape, &hp, &err)) return err;
    if (!mat_ok(k_score) || phi == nullptr || scores_out == nullptr) return COMPACTOR_E_INVALID_ARGUMENT;
    // Everything before the scores region must fit.  The fused sweep gets by with a shorter ring of Gram
    // partials (fewer pieces between the two reads of the keys); the separate kernels with longer Gram blocks.
    if (hp.fused) {
        while (hp.off_scores > kBuiltinScratchBytes && hp.window > hp.max_pieces + 1) {
            hp.window = hp.window / 2 > hp.max_pieces + 1 ? hp.window / 2 : hp.max_pieces + 1;
            layout_fused(&hp);
        }
    } else {
        while (hp.off_scores > kBuiltinScratchBytes && hp.plan.chunk < kMaxChunk) replan_chunk(shape, &hp, hp.plan.chunk * 2);
    }
    if (hp.off_scores > kBuiltinScratchBytes) return COMPACTOR_E_TOO_LARGE;
    if (hp.plan.total_tokens == 0) return COMPACTOR_OK;
    void* scratch = nullptr;
    int rc = builtin_scratch(&scratch);
    if (rc != COMPACTOR_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CK(upload_tables(&hp, scratch, st));
    return run_scoring(hp, to_mat(k_score), phi, attn_scores, lambda, scores_out, status,
                       static_cast<char*>(scratch), st);
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Token-averaged negative log-likelihood (Section 3.5).
extern "C" int compactor_nll(const void* logits, int32_t logits_dtype, int64_t rows, int32_t vocab, int64_t row_stride,
                             const int32_t* targets, int32_t batch, const int32_t* cu_rows, float* row_nll_out,
                             double* nll_out, void* stream) {
    if (logits_dtype != COMPACTOR_DTYPE_BF16 && logits_dtype != COMPACTOR_DTYPE_F32) return COMPACTOR_E_INVALID_ARGUMENT;
    if (rows < 0 || vocab < 1 || batch < 0 || cu_rows == nullptr || row_stride < vocab) return COMPACTOR_E_INVALID_ARGUMENT;
    if (cu_rows[0] != 0 || cu_rows[batch] != rows) return COMPACTOR_E_INVALID_ARGUMENT;
    for (int b = 0; b < batch; ++b)
        if (cu_rows[b + 1] < cu_rows[b]) return COMPACTOR_E_INVALID_ARGUMENT;
    if (batch == 0) return COMPACTOR_OK;
    if (nll_out == nullptr) return COMPACTOR_E_INVALID_ARGUMENT;
    if (rows > 0 && (logits == nullptr || targets == nullptr || row_nll_out == nullptr)) return COMPACTOR_E_INVALID_ARGUMENT;
    const size_t esize = logits_dtype == COMPACTOR_DTYPE_F32 ? 4 : 2;
    if (((uintptr_t)logits & 15) != 0 || ((size_t)row_stride * esize) % 16 != 0) return COMPACTOR_E_INVALID_ARGUMENT;
    CK(launch_nll(logits, logits_dtype == COMPACTOR_DTYPE_F32, rows, vocab, row_stride, targets, batch, cu_rows,
                  row_nll_out, nll_out, static_cast<cudaStream_t>(stream)));
    return COMPACTOR_OK;
}

// ---------------------------------------------------------------------------------------------
// Attention term (Eq. 5).
extern "C" int compactor_attention_scores_status(const compactor_shape* shape, compactor_mat q, compactor_mat k,
                                                 int32_t q_per_kv, int32_t chunk, float scale, int32_t pool,
                                                 float* attn_out, int32_t* status, void* workspace,
                                                 size_t workspace_bytes, void* stream) {
    HostPlan hp; int err = 0;
    if (!make_plan(shape, &hp, &err, false)) return err;
    if (chunk != 256) return COMPACTOR_E_UNSUPPORTED;
    if (!mat_ok(q) || !mat_ok(k) || attn_out == nullptr || workspace == nullptr || q_per_kv < 1 ||
        (long long)shape->heads * q_per_kv > 65535 || !(scale > 0.f) || !isfinite(scale) || pool < 1 || (pool & 1) == 0)
        return COMPACTOR_E_INVALID_ARGUMENT;
    if (((uintptr_t)workspace & 255) != 0) return COMPACTOR_E_INVALID_ARGUMENT;
    replan_chunk(shape, &hp, chunk);                 // one CTA per chunk of 256 tokens
    const size_t raw_bytes = pool > 1 ? sizeof(float) * (size_t)hp.plan.total_tokens * shape->layers * shape->heads : 0;
    if (workspace_bytes < hp.off_w + raw_bytes) return COMPACTOR_E_WORKSPACE;
    if (hp.plan.total_tokens == 0) return COMPACTOR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (status != nullptr) CK(cudaMemsetAsync(status, 0, sizeof(int32_t) * hp.units, st));
    CK(upload_tables(&hp, workspace, st));
    float* raw = reinterpret_cast<float*>(static_cast<char*>(workspace) + hp.off_w);
    CK(launch_attention(hp.plan, to_mat(q), to_mat(k), q_per_kv, scale, pool, raw, attn_out, status, st));
    return COMPACTOR_OK;
}

extern "C" int compactor_attention_scores(const compactor_shape* shape, compactor_mat q, compactor_mat k,
                                          int32_t q_per_kv, int32_t chunk, float scale, int32_t pool,
                                          float* attn_out, void* workspace, size_t workspace_bytes, void* stream) {
    return compactor_attention_scores_status(shape, q, k, q_per_kv, chunk, scale, pool, attn_out, nullptr, workspace,
                                             workspace_bytes, stream);
}

// ---------------------------------------------------------------------------------------------
// Selection across the heads of a layer and the matching gather.
extern "C" size_t compactor_across_heads_workspace_bytes(const compactor_shape* shape) {
    HostPlan hp; int err = 0;
    if (!make_plan(shape, &hp, &err)) return 0;
    return hp.off_w + across_scratch_bytes(shape, hp.plan.total_tokens);
}

extern "C" int compactor_select_across_heads(const compactor_shape* shape, const float* scores,
                                             const int32_t* keep_counts, int32_t* idx_out, int32_t* head_offsets_out,
                                             void* workspace, size_t workspace_bytes, void* stream) {
    HostPlan hp; int err = 0;
    if (!make_plan(shape, &hp, &err)) return err;
    if (shape->heads > 64) return COMPACTOR_E_UNSUPPORTED;
    if (scores == nullptr || idx_out == nullptr || head_offsets_out == nullptr || workspace == nullptr ||
        !set_keep(shape, keep_counts, &hp) || ((uintptr_t)workspace & 255) != 0)
        return COMPACTOR_E_INVALID_ARGUMENT;
    if ((long long)shape->heads * hp.plan.total_keep > 0x7fffffffLL) return COMPACTOR_E_INVALID_ARGUMENT;
    if (workspace_bytes < compactor_across_heads_workspace_bytes(shape)) return COMPACTOR_E_WORKSPACE;
    if (hp.plan.total_tokens == 0) return COMPACTOR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CK(upload_tables(&hp, workspace, st));
    CK(select_across(hp, shape, scores, idx_out, head_offsets_out, static_cast<char*>(workspace) + hp.off_w, st));
    return COMPACTOR_OK;
}

extern "C" int compactor_compact_across_heads(const compactor_shape* shape, compactor_mat k_cache, compactor_mat v_cache,
                                              const int32_t* idx, const int32_t* head_offsets,
                                              const int32_t* keep_counts, void* k_out, void* v_out,
                                              void* workspace, size_t workspace_bytes, void* stream) {
    HostPlan hp; int err = 0;
    if (!make_plan(shape, &hp, &err)) return err;
    if (!mat_ok(k_cache) || !mat_ok(v_cache) || idx == nullptr || head_offsets == nullptr || k_out == nullptr ||
        v_out == nullptr || workspace == nullptr || !set_keep(shape, keep_counts, &hp))
        return COMPACTOR_E_INVALID_ARGUMENT;
    if ((((uintptr_t)k_out | (uintptr_t)v_out) & 15) != 0 || ((uintptr_t)workspace & 255) != 0)
        return COMPACTOR_E_INVALID_ARGUMENT;
    if (workspace_bytes < hp.off_w) return COMPACTOR_E_WORKSPACE;
    if (hp.plan.total_keep == 0) return COMPACTOR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CK(upload_tables(&hp, workspace, st));
    CK(launch_compact_across(hp.plan, to_mat(k_cache), to_mat(v_cache), idx, head_offsets,
                             static_cast<__nv_bfloat16*>(k_out), static_cast<__nv_bfloat16*>(v_out), st));
    return COMPACTOR_OK;
}

// ---------------------------------------------------------------------------------------------
// The paper's whole method in one call (Sections 3.3, 3.4 and the set-up of Section 4).
namespace {

struct FullLayout {
    size_t off_attn, off_attn_ws, off_across, total;
    size_t main_bytes, attn_ws_bytes;
};

bool full_layout(const compactor_shape* shape, const compactor_options* opt, FullLayout* fl, int* err) {
    if (opt == nullptr) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    HostPlan hp;
    if (!make_plan(shape, &hp, err, false)) return false;
    if (opt->selection != COMPACTOR_SELECT_PER_HEAD && opt->selection != COMPACTOR_SELECT_ACROSS_HEADS) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    if (opt->factorization != COMPACTOR_FACTOR_CHOLESKY && opt->factorization != COMPACTOR_FACTOR_EIG) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    if (opt->q_per_kv < 0) { *err = COMPACTOR_E_INVALID_ARGUMENT; return false; }
    const size_t plane = sizeof(float) * (size_t)hp.plan.total_tokens * shape->layers * shape->heads;
    fl->main_bytes = compactor_workspace_bytes(shape);
    size_t off = align_up(fl->main_bytes);
    fl->off_attn = off;
    if (opt->q_per_kv > 0) off += align_up(plane);
    fl->off_attn_ws = off;
    fl->attn_ws_bytes = 0;
    if (opt->q_per_kv > 0) {
        fl->attn_ws_bytes = align_up(hp.off_w + (opt->pool > 1 ? plane : 0));
        off += fl->attn_ws_bytes;
    }
    fl->off_across = off;
    if (opt->selection == COMPACTOR_SELECT_ACROSS_HEADS) off += align_up(across_scratch_bytes(shape, hp.plan.total_tokens));
    fl->total = off;
    return true;
}

}  // namespace

extern "C" size_t compactor_compress_full_workspace_bytes(const compactor_shape* shape, const compactor_options* options) {
    FullLayout fl; int err = 0;
    if (!full_layout(shape, options, &fl, &err)) return 0;
    return fl.total;
}

extern "C" int compactor_compress_full(const compactor_shape* shape, const compactor_options* options, compactor_mat q,
                                       compactor_mat k_score, compactor_mat k_cache, compactor_mat v_cache,
                                       const float* phi, const int32_t* keep_counts, float* scores_out,
                                       int32_t* idx_out, int32_t* head_offsets_out, void* k_out, void* v_out,
                                       int32_t* status, void* workspace, size_t workspace_bytes, void* stream) {
    FullLayout fl; int err = 0;
    if (!full_layout(shape, options, &fl, &err)) return err;
    const bool across = options->selection == COMPACTOR_SELECT_ACROSS_HEADS;
    const bool with_attn = options->q_per_kv > 0;
    const bool eig = options->factorization == COMPACTOR_FACTOR_EIG;
    HostPlan hp;
    if (!make_plan(shape, &hp, &err, !eig)) return err;
    if (eig && (hp.plan.mp > 64 || !(options->eig_floor > 0.0) || !std::isfinite(options->eig_floor)))
        return hp.plan.mp > 64 ? COMPACTOR_E_UNSUPPORTED : COMPACTOR_E_INVALID_ARGUMENT;
    if (!mat_ok(k_score) || !mat_ok(k_cache) || !mat_ok(v_cache) || phi == nullptr || idx_out == nullptr ||
        k_out == nullptr || v_out == nullptr || workspace == nullptr || !set_keep(shape, keep_counts, &hp))
        return COMPACTOR_E_INVALID_ARGUMENT;
    if ((((uintptr_t)k_out | (uintptr_t)v_out) & 15) != 0 || ((uintptr_t)workspace & 255) != 0)
        return COMPACTOR_E_INVALID_ARGUMENT;
    if (across && (head_offsets_out == nullptr || (long long)shape->heads * hp.plan.total_keep > 0x7fffffffLL))
        return COMPACTOR_E_INVALID_ARGUMENT;
    if (across && shape->heads > 64) return COMPACTOR_E_UNSUPPORTED;
    if (with_attn) {
        if (options->chunk != 256) return COMPACTOR_E_UNSUPPORTED;
        if (!mat_ok(q) || (long long)shape->heads * options->q_per_kv > 65535 || !(options->scale > 0.f) ||
            !isfinite(options->scale) || options->pool < 1 || (options->pool & 1) == 0)
            return COMPACTOR_E_INVALID_ARGUMENT;
    }
    if (workspace_bytes < fl.total) return COMPACTOR_E_WORKSPACE;
    if (hp.plan.total_tokens == 0) return COMPACTOR_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    if (status != nullptr) CK(cudaMemsetAsync(status, 0, sizeof(int32_t) * hp.units, st));
    float* attn = nullptr;
    if (with_attn) {
        // Eq. 5 on the cache's keys (the ones attention sees), into a plane of the workspace
        HostPlan ap;
        if (!make_plan(shape, &ap, &err, false)) return err;
        replan_chunk(shape, &ap, options->chunk);
        char* aws = ws + fl.off_attn_ws;
        CK(upload_tables(&ap, aws, st));
        attn = reinterpret_cast<float*>(ws + fl.off_attn);
        CK(launch_attention(ap.plan, to_mat(q), to_mat(k_cache), options->q_per_kv, options->scale, options->pool,
                            reinterpret_cast<float*>(aws + ap.off_w), attn, status, st));
    }
    float* scores = scores_out != nullptr ? scores_out : reinterpret_cast<float*>(ws + hp.off_scores);
    CK(upload_tables(&hp, ws, st));
    const int rc = run_scoring(hp, to_mat(k_score), phi, attn, options->lambda, scores, status, ws, st, Marks(),
                               options->factorization, options->eig_floor, false);
    if (rc != COMPACTOR_OK) return rc;
    if (!across) {
        if (hp.plan.total_keep > 0) {
            CK(select_per_head(hp, shape, scores, idx_out, ws + hp.off_w, hp.off_scores - hp.off_w, st));
            CK(launch_compact(hp.plan, to_mat(k_cache), to_mat(v_cache), idx_out,
                              static_cast<__nv_bfloat16*>(k_out), static_cast<__nv_bfloat16*>(v_out), st));
        }
    } else {
        CK(select_across(hp, shape, scores, idx_out, head_offsets_out, ws + fl.off_across, st));
        if (hp.plan.total_keep > 0)
            CK(launch_compact_across(hp.plan, to_mat(k_cache), to_mat(v_cache), idx_out, head_offsets_out,
                                     static_cast<__nv_bfloat16*>(k_out), static_cast<__nv_bfloat16*>(v_out), st));
    }
    return COMPACTOR_OK;
}

// ---------------------------------------------------------------------------------------------
// Appendix D: the subsampled randomised Hadamard sketch as an explicit matrix (host helper).
extern "C" int compactor_make_sketch_srht(uint64_t seed, int32_t d, int32_t m, float* phi_host) {
    if (phi_host == nullptr || d < 1 || (d & (d - 1)) != 0 || m < 1 || m > d) return COMPACTOR_E_INVALID_ARGUMENT;
    auto word = [seed](uint64_t i) {
        uint64_t z = seed + (i + 1) * 0x9E3779B97F4A7C15ull;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        return z ^ (z >> 31);
    };
    std::vector<int> perm(d);
    for (int i = 0; i < d; ++i) perm[i] = i;
    for (int j = 0; j < m; ++j) {
        const int r = j + (int)(word((uint64_t)d + j) % (uint64_t)(d - j));
        const int tmp = perm[j]; perm[j] = perm[r]; perm[r] = tmp;
    }
    const float mag = (float)(1.0 / sqrt((double)m));
    for (int i = 0; i < d; ++i) {
        const bool minus_row = (word((uint64_t)i) & 1ull) != 0;
        for (int j = 0; j < m; ++j) {
            const bool minus_h = (__builtin_popcount((unsigned)(i & perm[j])) & 1) != 0;   // Sylvester: H[i][c] = (-1)^popcount(i & c)
            phi_host[(size_t)i * m + j] = (minus_row != minus_h) ? -mag : mag;
        }
    }
    return COMPACTOR_OK;
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded waits.  Every spin of the streaming kernels goes through
// sm100::mbar_wait, which gives up after a cycle limit and lets the kernel report
// COMPACTOR_STATUS_TIMEOUT instead of hanging the device.  This entry point runs that same wait on
// a barrier that nothing will ever complete, with a limit of about one millisecond, and writes what
// the wait returned, so that the give-up path can be exercised without faulting or hanging a GPU.
namespace {
__global__ void wait_selftest_kernel(int* status_out, long long limit_cycles) {
    __shared__ uint64_t never;
    __shared__ uint64_t once;
    if (threadIdx.x == 0) {
        compactor::sm100::mbar_init(&never, 1);
        compactor::sm100::mbar_init(&once, 1);
        compactor::sm100::fence_barrier_init();
        compactor::sm100::mbar_arrive(&once);                                  // this one does complete
        const bool completed = compactor::sm100::mbar_wait(&once, 0, limit_cycles);
        const bool hung = compactor::sm100::mbar_wait(&never, 0, limit_cycles);   // runs out
        status_out[0] = (completed ? 0 : 8) | (hung ? 0 : COMPACTOR_STATUS_TIMEOUT);
    }
}
}  // namespace

extern "C" int compactor_wait_selftest(int32_t* status_out, void* stream) {
    if (status_out == nullptr) return COMPACTOR_E_INVALID_ARGUMENT;
    wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status_out, 2000000LL);
    return cudaGetLastError() == cudaSuccess ? COMPACTOR_OK : COMPACTOR_E_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Section 3.5: fit of the calibration curve's two parameters (host helper).
namespace {

double curve(double r, double b) {                  // f(r) = (e^{br} - 1) / (e^b - 1), f = r at b = 0
    if (fabs(b) < 1e-8) return r + 0.5 * b * r * (r - 1.0);
    return expm1(b * r) / expm1(b);
}
double curve_db(double r, double b) {               // d f / d b
    if (fabs(b) < 1e-4) return 0.5 * r * (r - 1.0) + b * r * (r - 1.0) * (2.0 * r - 1.0) / 6.0;
    const double eb = expm1(b), er = expm1(b * r);
    return (r * (er + 1.0) * eb - er * (eb + 1.0)) / (eb * eb);
}
double fit_loss(long long n, const double* r, const double* c, const double* y, double w_under, double al, double be) {
    double s = 0.0;
    for (long long i = 0; i < n; ++i) {
        const double e = curve(r[i], al * c[i] + be) - y[i];
        s += (e > 0.0 ? w_under : 1.0) * e * e;
    }
    return s / (double)n;
}

}  // namespace

extern "C" int compactor_fit_calibration(int64_t n, const double* r, const double* nll, const double* y,
                                         double under_weight, double* alpha_out, double* beta_out, double* loss_out) {
    if (n < 2 || r == nullptr || nll == nullptr || y == nullptr || alpha_out == nullptr || beta_out == nullptr ||
        !(under_weight >= 1.0))
        return COMPACTOR_E_INVALID_ARGUMENT;
    double best = 1e300, best_a = 0.0, best_b = 0.0;
    const double a_starts[4] = {-4.0, -1.0, 0.0, 1.0}, b_starts[3] = {-6.0, -2.0, 0.5};
    for (double a0 : a_starts)
        for (double b0 : b_starts) {
            // Levenberg-Marquardt on (alpha, beta); the asymmetric weights are those of the current residuals
            double al = a0, be = b0, mu = 1e-3, cur = fit_loss(n, r, nll, y, under_weight, al, be);
            for (int iter = 0; iter < 500; ++iter) {
                double jaa = 0, jab = 0, jbb = 0, ga = 0, gb = 0;
                for (long long i = 0; i < n; ++i) {
                    const double b = al * nll[i] + be;
                    const double e = curve(r[i], b) - y[i];
                    const double w = e > 0.0 ? under_weight : 1.0;
                    const double db = curve_db(r[i], b), da = db * nll[i];
                    jaa += w * da * da; jab += w * da * db; jbb += w * db * db;
                    ga += w * da * e; gb += w * db * e;
                }
                bool improved = false;
                for (int tries = 0; tries < 30 && !improved; ++tries) {
                    const double haa = jaa * (1.0 + mu) + 1e-300, hbb = jbb * (1.0 + mu) + 1e-300;
                    const double det = haa * hbb - jab * jab;
                    if (!(fabs(det) > 0.0)) { mu *= 10.0; continue; }
                    const double sa = -(hbb * ga - jab * gb) / det, sb = -(haa * gb - jab * ga) / det;
                    const double trial = fit_loss(n, r, nll, y, under_weight, al + sa, be + sb);
                    if (trial < cur) {
                        al += sa; be += sb; improved = true;
                        const bool tiny = fabs(sa) + fabs(sb) < 1e-13 || cur - trial < 1e-18 * (1.0 + cur);
                        cur = trial; mu = fmax(mu * 0.3, 1e-12);
                        if (tiny) iter = 500;
                    } else {
                        mu *= 10.0;
                    }
                }
                if (!improved) break;
            }
            if (cur < best) { best = cur; best_a = al; best_b = be; }
        }
    *alpha_out = best_a; *beta_out = best_b;
    if (loss_out != nullptr) *loss_out = best;
    return COMPACTOR_OK;
}
