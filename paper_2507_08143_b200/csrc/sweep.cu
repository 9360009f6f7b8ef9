// Fused scoring sweep (Algorithm 1, lines 2-6) as ONE persistent kernel: Gram pieces, the small
// factorisation and the scoring pieces of all units run from a common, dependency-driven work
// queue, so that the second read of a unit's keys (line 5, after line 3) finds them in L2.
//
// Work decomposition.  Every unit's tokens are cut into pieces of `chunk` tokens (1024 unless a
// sequence is very long).  A piece is visited twice:
//   Gram piece    C_p = K_p^T K_p on tcgen05 (fp32 in tensor memory over at most 512 tokens, fp64
//                 in registers beyond), stored as one fp32 128 x 128 partial in a ring of slots.
//   scoring piece o_i = || k_i W ||^2 with W = Phi L^-T of the unit, as two bf16 terms, one
//                 tcgen05.mma per k-step, fused square-and-sum epilogue.
// Between the two sits the unit's factorisation, cut into `slices` row slices:
//   slice task    rows of C = sum of the unit's partials (fp64, fixed order), T = C[rows] Phi as
//                 fp64 mma.m8n8k4; the CTA that finishes a unit's last slice goes on with
//                 G = Phi^T T, the Cholesky factor G = L L^T (pivots below 2^-20 of their
//                 diagonal entry dropped: pseudo-inverse reading) and W = Phi L^-T.
//
// Scheduling.  One CTA per SM.  Warp 10 claims sweep pieces from global counters (a scoring piece
// whose W is ready first, else the next Gram piece, which may run at most `window` pieces ahead of
// the scoring front: that bounds the keys waiting in L2) and hands them, through a small queue, to
// warp 0 (which streams their tiles through a ring of shared memory with TMA), warp 1 (tcgen05.mma
// issue) and warps 2-9 (epilogue).  Between pieces, and whenever they are idle, warps 2-9 claim factor tasks.
// Claims are fetch-adds on per-unit counters (they never fail, so any number of CTAs can claim at once);
// two 64-bit words hold, each, the prefix of units that are ready and the prefix that is used up, and
// move by compare-and-swap once per unit.  Results do not depend on who runs what: every sum has a
// fixed order and every piece a fixed slot.
//
// Every wait is bounded.  When one runs out the CTA raises its abort flag and a global one, all
// further waits fall through (control flow stays the same, so no thread is left at a barrier),
// and the unit is flagged COMPACTOR_STATUS_TIMEOUT.
#include "common.cuh"
#include "factor_math.cuh"
#include "sm100.cuh"

namespace compactor {
namespace {

using namespace sm100;
using namespace factor_math;

constexpr int kTile = 128;
constexpr int kBoxBytes = kTile * 128;     // 64 channels x 128 tokens x 2 B
constexpr int kTileBytes = 2 * kBoxBytes;
constexpr int kStages = 4;
constexpr int kFlushTiles = kGramFlushTokens / kTile;
constexpr int kWorkerWarps = 8;
constexpr int kWorkers = 32 * kWorkerWarps;
constexpr int kThreads = 64 + kWorkers + 32;   // warp 0: TMA loads, warp 1: MMA, warps 2-9: epilogue and factor tasks, warp 10: scheduler
constexpr int kSchedWarp = 2 + kWorkerWarps;
constexpr int kQueue = 3;                  // pieces handed over inside a CTA (the scheduler claims at most this far ahead)
constexpr uint32_t kTmemCols = 512;        // two Gram accumulators (128 columns each) + two scoring accumulators
constexpr uint32_t kScoreCol0 = 256;
constexpr int kOutTiles = 4;               // tiles whose scores leave together
constexpr int kExactGramTokens = 256;      // units this short take their Gram matrix in fp64 straight from the keys
constexpr int kStageTokens = 8;
constexpr int kLdC = kD + 4;               // row stride (doubles) of the staged rows of C: fragment loads without bank conflicts

#ifdef COMPACTOR_SWEEP_PROFILE
#define PROF_T(var) const long long var = clock64()
#define PROF_ADD(slot, t_begin) do { if (a.prof != nullptr) a.prof[blockIdx.x * 32 + (slot)] += clock64() - (t_begin); } while (0)
#define PROF_INC(slot) do { if (a.prof != nullptr) a.prof[blockIdx.x * 32 + (slot)] += 1; } while (0)
#else
#define PROF_T(var) do {} while (0)
#define PROF_ADD(slot, t_begin) do {} while (0)
#define PROF_INC(slot) do {} while (0)
#endif

enum { kTaskGram = 0, kTaskScore = 1, kTaskExit = 2 };
enum { kActSweep = 0, kActFactor = 1, kActQuit = 2 };

struct Task { int type, piece, lh, b, tok_begin, n_tok, unit, pad; };

template <int MP>
struct __align__(1024) SweepSmem {
    static constexpr int kLd = MP;         // column stride of G and L (doubles)
    static constexpr int kLdT = MP + 4;    // row stride of a staged block of T
    unsigned char tiles[kStages][kTileBytes];
    unsigned char w[2][2][2][MP * 128];    // [buffer][channel half][term][MP rows x 64 channels]
    float phi[kD * MP];                    // the sketch, zero in the padded columns
    union Scratch {
        struct { double c[8 * kLdC]; double keys[kStageTokens * kD]; } slice;
        double t[kTRows * kLdT];
        struct { double g[MP * kLd]; double diag0[MP]; double inv_diag[MP]; } chol;
    } scratch;
    float obuf[2][kOutTiles * kTile];
    Task tq[kQueue];
    uint64_t full[kStages], empty[kStages];
    uint64_t gacc_full[2], gacc_empty[2], sacc_full[2], sacc_empty[2];
    uint64_t w_full[2], w_empty[2];
    uint64_t tq_full[kQueue], tq_empty[kQueue];
    uint32_t tmem_base;
    int abort;
    int w_action[2], w_arg[2], w_arg2[2];
    int flags, last;
};

// ------------------------------------------------------------------ global-memory synchronisation
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_release_u32(unsigned* p, unsigned v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void workers_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kWorkers) : "memory"); }

__device__ __forceinline__ int unit_pieces(const Plan& p, int unit) {
    const int b = unit % p.batch;
    return p.cu_chunks[b + 1] - p.cu_chunks[b];
}
__device__ __forceinline__ int unit_piece_start(const Plan& p, int unit) {
    const int lh = unit / p.batch, b = unit - lh * p.batch;
    return lh * p.total_chunks + p.cu_chunks[b];
}
__device__ __forceinline__ void piece_to_task(const Plan& p, int piece, int type, Task* t) {
    const int lh = piece / p.total_chunks, c = piece - lh * p.total_chunks;
    const int b = find_segment(p.cu_chunks, p.batch, c);
    const int tok_begin = p.cu_seqlens[b] + (c - p.cu_chunks[b]) * p.chunk;
    t->type = type; t->piece = piece; t->lh = lh; t->b = b; t->tok_begin = tok_begin;
    t->n_tok = min(p.chunk, p.cu_seqlens[b + 1] - tok_begin);
    t->unit = lh * p.batch + b; t->pad = 0;
}

// Moves the "Gram complete" prefix of units forward as far as it goes.
__device__ void advance_gram_prefix(const SweepArgs& a) {
    for (;;) {
        const unsigned long long fs = ld_acquire_u64(&a.sched->fstate);
        const unsigned gu = (unsigned)fs;
        if ((int)gu >= a.units) return;
        if ((int)ld_acquire_u32(reinterpret_cast<const unsigned*>(a.gram_done) + gu) != unit_pieces(a.p, (int)gu)) return;
        __threadfence();
        atomicCAS(&a.sched->fstate, fs, fs + 1ull);
    }
}
// The same for the prefix of units whose W is written.
__device__ void advance_w_prefix(const SweepArgs& a) {
    for (;;) {
        const unsigned long long ss = ld_acquire_u64(&a.sched->sstate);
        const unsigned wu = (unsigned)ss;
        if ((int)wu >= a.units) return;
        if (ld_acquire_u32(reinterpret_cast<const unsigned*>(a.w_ready) + wu) == 0u) return;
        __threadfence();
        atomicCAS(&a.sched->sstate, ss, ss + 1ull);
    }
}

template <int MP>
__global__ void __launch_bounds__(kThreads, 1)
sweep_kernel(const __grid_constant__ SweepArgs a, const __grid_constant__ CUtensorMap kmap,
             const __grid_constant__ CUtensorMap wmap) {
    extern __shared__ unsigned char smem_raw[];
    using Smem = SweepSmem<MP>;
    Smem& s = *reinterpret_cast<Smem*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
    const Plan& p = a.p;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_pieces = a.total_pieces;

    if (threadIdx.x == 0) {
        prefetch_tensormap(&kmap);
        prefetch_tensormap(&wmap);
        for (int i = 0; i < kStages; ++i) { mbar_init(&s.full[i], 1); mbar_init(&s.empty[i], 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s.gacc_full[i], 1); mbar_init(&s.gacc_empty[i], kWorkerWarps);
            mbar_init(&s.sacc_full[i], 1); mbar_init(&s.sacc_empty[i], kWorkerWarps / 2);
            mbar_init(&s.w_full[i], 1);    mbar_init(&s.w_empty[i], 1);
        }
        for (int i = 0; i < kQueue; ++i) { mbar_init(&s.tq_full[i], 1); mbar_init(&s.tq_empty[i], 2 + kWorkerWarps); }
        s.abort = 0;
        fence_barrier_init();
    }
    for (int i = threadIdx.x; i < kD * MP; i += kThreads) {
        const int row = i / MP, col = i - row * MP;
        s.phi[i] = col < p.m ? __ldg(a.phi + row * p.m + col) : 0.f;
    }
    if (warp == 1) { tmem_alloc(&s.tmem_base, kTmemCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = s.tmem_base;

    // A wait that gives up: afterwards every wait of this CTA falls through.
    auto wait = [&](uint64_t* bar, uint32_t parity) {
        if (*(volatile int*)&s.abort) return;
        if (!mbar_wait(bar, parity)) { s.abort = 1; atomicExch(&a.sched->abort, 1u); }
    };
    int last_unit = 0;

    if (warp == kSchedWarp) {
        // ------------------------------------------------------------ scheduler: claims pieces, ahead of the loads
        if (lane == 0) {
            int tq_count = 0;
            for (;;) {
                Task t;
                t.type = kTaskExit; t.piece = 0; t.lh = 0; t.b = 0; t.tok_begin = 0; t.n_tok = 0; t.unit = 0; t.pad = 0;
                const long long t0 = clock64();
                for (;;) {
                    PROF_INC(1);
                    if (*(volatile int*)&s.abort || *(volatile unsigned*)&a.sched->abort) break;
                    const unsigned long long ss = ld_acquire_u64(&a.sched->sstate);
                    const unsigned g = *(volatile unsigned*)&a.sched->gram_next;
                    const int s_unit = (int)(ss >> 32);
                    const int w_units = a.phase == 2 ? a.units : (int)(unsigned)ss;     // the scoring launch finds every W written
                    if (s_unit >= a.units) break;                      // every scoring piece has been claimed
                    if (a.phase == 1 && (int)g >= total_pieces) break; // the Gram launch: every Gram piece has been claimed
                    if (a.phase != 1 && s_unit < w_units) {
                        // a scoring piece of the first unit that still has some: claims are fetch-adds, they never fail
                        const int idx = atomicAdd(a.score_claimed + s_unit, 1);
                        if (idx < unit_pieces(p, s_unit)) {
                            piece_to_task(p, unit_piece_start(p, s_unit) + idx, kTaskScore, &t);
                            break;
                        }
                        atomicCAS(&a.sched->sstate, ss, ss + (1ull << 32));     // the unit is used up: move on
                        continue;
                    }
                    if (w_units < a.units && ld_acquire_u32(reinterpret_cast<const unsigned*>(a.w_ready) + w_units) != 0u) {
                        __threadfence();
                        atomicCAS(&a.sched->sstate, ss, ss + 1ull);
                        continue;
                    }
                    // Gram pieces may run `window` pieces ahead of the scoring front (of the units whose W is written, in
                    // the launch that does no scoring): their partial sums live in a ring of slots
                    const int front = a.phase == 1 ? w_units : s_unit;
                    if (a.phase != 2 && (int)g < total_pieces &&
                        (int)g < (front >= a.units ? total_pieces : unit_piece_start(p, front)) + a.window) {
                        const int idx = (int)atomicAdd(&a.sched->gram_next, 1u);
                        if (idx < total_pieces) { piece_to_task(p, idx, kTaskGram, &t); break; }
                        continue;
                    }
                    __nanosleep(200);
                    if (clock64() - t0 > kWaitLimitCycles) { s.abort = 1; atomicExch(&a.sched->abort, 1u); break; }
                }
                PROF_ADD(0, t0);
                PROF_T(tp1);
                const int slot = tq_count % kQueue, qround = tq_count / kQueue;
                if (qround > 0) wait(&s.tq_empty[slot], (qround - 1) & 1);
                PROF_ADD(2, tp1);
                if (t.type == kTaskGram) PROF_INC(3);
                if (t.type == kTaskScore) PROF_INC(4);
                s.tq[slot] = t;
                mbar_arrive(&s.tq_full[slot]);
                ++tq_count;
                if (t.type == kTaskExit) break;
            }
        }
    } else if (warp == 0) {
        // ------------------------------------------------------------ TMA loads of the claimed pieces
        if (lane == 0) {
            uint64_t pol_first;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_first));
            int tq_count = 0, tile_count = 0, score_count = 0;
            for (;;) {
                const int slot = tq_count % kQueue;
                wait(&s.tq_full[slot], (tq_count / kQueue) & 1);
                const Task t = s.tq[slot];
                ++tq_count;
                if (t.type == kTaskExit) { mbar_arrive(&s.tq_empty[slot]); break; }
                last_unit = t.unit;
                const int layer = t.lh / p.heads, head = t.lh - layer * p.heads;
                if (t.type == kTaskScore) {
                    const int wb = score_count & 1;
                    if (score_count >= 2) wait(&s.w_empty[wb], ((score_count >> 1) - 1) & 1);
                    if (!*(volatile int*)&s.abort) {
                        asm volatile("fence.proxy.async;" ::: "memory");      // W was written with ordinary stores by another SM
                        mbar_arrive_expect_tx(&s.w_full[wb], 4 * MP * 128);
#pragma unroll
                        for (int term = 0; term < 2; ++term)
#pragma unroll
                            for (int half = 0; half < 2; ++half)
                                tma_load_2d(s.w[wb][half][term], &wmap, &s.w_full[wb], half * 64, (t.unit * 2 + term) * MP);
                    }
                    ++score_count;
                }
                // Keys that are to wait in L2 for their second read are loaded with the default priority; the second
                // read itself, and the first read of the pieces that are not meant to stay, leave first.
                const int in_unit = t.piece - unit_piece_start(p, t.unit);
                const bool stays = t.type == kTaskGram && ((in_unit * 5) & 15) < a.resident16;
                const int n_tiles = (t.n_tok + kTile - 1) / kTile;
                PROF_T(tp2);
                for (int j = 0; j < n_tiles; ++j) {
                    const int stage = tile_count % kStages, round = tile_count / kStages;
                    if (round > 0) wait(&s.empty[stage], (round - 1) & 1);
                    ++tile_count;
                    if (*(volatile int*)&s.abort) continue;
                    mbar_arrive_expect_tx(&s.full[stage], kTileBytes);
                    const int tok = t.tok_begin + j * kTile;
                    if (!stays) {
                        tma_load_4d_hint(s.tiles[stage], &kmap, &s.full[stage], 0, tok, head, layer, pol_first);
                        tma_load_4d_hint(s.tiles[stage] + kBoxBytes, &kmap, &s.full[stage], 64, tok, head, layer, pol_first);
                    } else {
                        tma_load_4d(s.tiles[stage], &kmap, &s.full[stage], 0, tok, head, layer);
                        tma_load_4d(s.tiles[stage] + kBoxBytes, &kmap, &s.full[stage], 64, tok, head, layer);
                    }
                }
                PROF_ADD(t.type == kTaskGram ? 5 : 6, tp2);
                mbar_arrive(&s.tq_empty[slot]);
            }
            // After a give-up some copies may still be on their way into this CTA's shared memory.
            if (*(volatile int*)&s.abort) {
                for (int back = 1; back <= kStages && back <= tile_count; ++back) {
                    const int tc = tile_count - back;
                    mbar_wait(&s.full[tc % kStages], (tc / kStages) & 1);
                }
                for (int back = 1; back <= 2 && back <= score_count; ++back) {
                    const int sc = score_count - back;
                    mbar_wait(&s.w_full[sc & 1], (sc >> 1) & 1);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ tcgen05.mma issue
        constexpr uint32_t idesc_gram = umma_idesc_bf16(128, 128, 1, 1);
        constexpr uint32_t idesc_score = umma_idesc_bf16(128, 2 * MP, 0, 0);
        int tq_count = 0, tile_count = 0, g_groups = 0, s_tiles = 0, score_count = 0;
        for (;;) {
            const int slot = tq_count % kQueue;
            PROF_T(tm0);
            wait(&s.tq_full[slot], (tq_count / kQueue) & 1);
            if (lane == 0) PROF_ADD(23, tm0);
            const Task t = s.tq[slot];
            ++tq_count;
            if (t.type == kTaskExit || *(volatile int*)&s.abort) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&s.tq_empty[slot]);
                if (t.type == kTaskExit) break;
                continue;
            }
            const int n_tiles = (t.n_tok + kTile - 1) / kTile;
            if (t.type == kTaskGram) {
                for (int j = 0; j < n_tiles; ++j) {
                    const int stage = tile_count % kStages, round = tile_count / kStages;
                    ++tile_count;
                    const int gg = g_groups + j / kFlushTiles, in_group = j % kFlushTiles, buf = gg & 1;
                    PROF_T(tm1);
                    if (in_group == 0 && gg >= 2) wait(&s.gacc_empty[buf], ((gg >> 1) - 1) & 1);
                    if (lane == 0) PROF_ADD(24, tm1);
                    PROF_T(tm2);
                    wait(&s.full[stage], round & 1);
                    if (lane == 0) PROF_ADD(25, tm2);
                    tc_fence_after_sync();
                    const int valid = min(kTile, t.n_tok - j * kTile);
                    if (valid < kTile) {
                        // rows past the end of the sequence belong to someone else (or to nobody): clear them
                        const int rows = kTile - valid;
                        for (int i = lane; i < rows * 16; i += 32) {
                            const int box = i / (rows * 8), jj = i % (rows * 8);
                            const int row = valid + (jj >> 3), piece16 = jj & 7;
                            *reinterpret_cast<uint4*>(s.tiles[stage] + box * kBoxBytes + row * 128 + piece16 * 16) =
                                make_uint4(0, 0, 0, 0);
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                    }
                    if (lane == 0) {
                        const uint32_t base = smem_u32(s.tiles[stage]);
                        const uint32_t d_addr = tmem + buf * 128;
#pragma unroll
                        for (int ks = 0; ks < kTile / 16; ++ks) {
                            const uint64_t desc = umma_desc_sw128(base + ks * 2048, kBoxBytes, 1024);
                            umma_bf16(d_addr, desc, desc, idesc_gram, (in_group > 0) || (ks > 0));
                        }
                        umma_commit(&s.empty[stage]);
                        if (in_group == kFlushTiles - 1 || j == n_tiles - 1) umma_commit(&s.gacc_full[buf]);
                    }
                    __syncwarp();
                }
                g_groups += (n_tiles + kFlushTiles - 1) / kFlushTiles;
            } else {
                const int wb = score_count & 1;
                PROF_T(tm3);
                wait(&s.w_full[wb], (score_count >> 1) & 1);
                if (lane == 0) PROF_ADD(26, tm3);
                for (int j = 0; j < n_tiles; ++j) {
                    const int stage = tile_count % kStages, round = tile_count / kStages;
                    ++tile_count;
                    const int buf = s_tiles & 1, use = s_tiles >> 1;
                    ++s_tiles;
                    PROF_T(tm4);
                    wait(&s.full[stage], round & 1);
                    if (lane == 0) PROF_ADD(27, tm4);
                    PROF_T(tm5);
                    if (use > 0) wait(&s.sacc_empty[buf], (use - 1) & 1);
                    if (lane == 0) PROF_ADD(28, tm5);
                    tc_fence_after_sync();
                    if (lane == 0) {
                        const uint32_t a_base = smem_u32(s.tiles[stage]);
                        const uint32_t d_addr = tmem + kScoreCol0 + buf * 128;
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            const int half = ks >> 2, off = (ks & 3) * 32;
                            const uint64_t a_desc = umma_desc_sw128(a_base + half * kBoxBytes + off, 16, 1024);
                            const uint64_t b_desc = umma_desc_sw128(smem_u32(s.w[wb][half][0]) + off, 16, 1024);
                            umma_bf16(d_addr, a_desc, b_desc, idesc_score, ks > 0);
                        }
                        umma_commit(&s.empty[stage]);
                        umma_commit(&s.sacc_full[buf]);
                    }
                    __syncwarp();
                }
                if (lane == 0) umma_commit(&s.w_empty[wb]);
                ++score_count;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&s.tq_empty[slot]);
        }
    } else if (warp >= 2 && warp < kSchedWarp) {
        // ------------------------------------------------------------ epilogue warps and factor tasks
        const int wtid = threadIdx.x - 64, wwarp = warp - 2;
        const int q = warp & 3;                          // TMEM lane quadrant this warp may read
        const int fr = lane >> 2, fk = lane & 3;         // fp64 mma fragment coordinates
        int tq_count = 0, g_groups = 0, s_tiles = 0, iter = 0;
        unsigned long long hint_fs = 0;
        bool have_hint = false;
        bool draining = false;       // the Gram launch: no pieces left for this CTA, but factor tasks may still come
        for (;;) {
            // ---- the leader picks the next thing to do: a factor task that is ready, else the next piece of this CTA
            PROF_T(tw0);
            if (wtid == 0) {
                int action = kActSweep, arg = 0, arg2 = 0;
                const int slot = tq_count % kQueue;
                const uint32_t qphase = (tq_count / kQueue) & 1;
                const long long t0 = clock64();
                for (;;) {
                    if (*(volatile int*)&s.abort) {
                        if (draining) { action = kActQuit; break; }
                        // the scheduler stops claiming and hands over the exit task: wait for it (short, bounded)
                        if (mbar_try_wait(&s.tq_full[slot], qphase) || clock64() - t0 > kWaitLimitCycles) break;
                        continue;
                    }
                    const unsigned long long fs = have_hint ? hint_fs : ld_acquire_u64(&a.sched->fstate);
                    const bool fresh = !have_hint;
                    have_hint = false;
                    const int f_unit = (int)(fs >> 32), gunits = (int)(unsigned)fs;
                    if (f_unit < gunits) {
                        const int fb = f_unit % p.batch;
                        const int idx = atomicAdd(a.slices_claimed + f_unit, 1);
                        if (idx < p.cu_schunks[fb + 1] - p.cu_schunks[fb]) {
                            __threadfence();
                            action = kActFactor; arg = f_unit; arg2 = idx;
                            break;
                        }
                        atomicCAS(&a.sched->fstate, fs, fs + (1ull << 32));     // all slices of that unit are taken: move on
                        continue;
                    }
                    if (draining) {
                        if (f_unit >= a.units || *(volatile unsigned*)&a.sched->abort) { action = kActQuit; break; }
                    } else if (mbar_try_wait(&s.tq_full[slot], qphase)) break;
                    if (!fresh) continue;                 // the hint was old: look again before sleeping
                    if (gunits < a.units &&
                        (int)ld_acquire_u32(reinterpret_cast<const unsigned*>(a.gram_done) + gunits) == unit_pieces(p, gunits)) {
                        __threadfence();
                        atomicCAS(&a.sched->fstate, fs, fs + 1ull);
                        continue;
                    }
                    __nanosleep(100);
                    if (clock64() - t0 > kWaitLimitCycles) { s.abort = 1; atomicExch(&a.sched->abort, 1u); }
                }
                s.w_action[iter & 1] = action;
                s.w_arg[iter & 1] = arg;
                s.w_arg2[iter & 1] = arg2;
            }
            workers_sync();
            const int action = s.w_action[iter & 1], arg = s.w_arg[iter & 1], arg2 = s.w_arg2[iter & 1];
            ++iter;
            if (wtid == 0) PROF_ADD(8, tw0);
            PROF_T(tw1);

            if (action == kActQuit) break;
            if (action == kActSweep) {
                const int slot = tq_count % kQueue;
                const Task t = s.tq[slot];
                ++tq_count;
                if (t.type == kTaskExit) {
                    if (a.phase != 1) break;
                    draining = true;          // stay for the factor tasks of the units that are still being summed
                    continue;
                }
                if (wtid == 0) { hint_fs = ld_relaxed_u64(&a.sched->fstate); have_hint = true; }
                const int n_tiles = (t.n_tok + kTile - 1) / kTile;
                if (t.type == kTaskGram) {
                    // ---- Gram epilogue: 64 columns of one row of C per thread, fp64 across the 512-token runs
                    const int half = wwarp >> 2;
                    const int row = q * 32 + lane;
                    const int n_groups = (n_tiles + kFlushTiles - 1) / kFlushTiles;
                    double acc[64];
#pragma unroll
                    for (int i = 0; i < 64; ++i) acc[i] = 0.0;
                    for (int g = 0; g < n_groups; ++g) {
                        const int gg = g_groups + g, buf = gg & 1;
                        wait(&s.gacc_full[buf], (gg >> 1) & 1);
                        tc_fence_after_sync();
#pragma unroll
                        for (int c0 = 0; c0 < 64; c0 += 32) {
                            uint32_t r[32];
                            tmem_ld_32x32b_x32(tmem + ((uint32_t)(q * 32) << 16) + buf * 128 + half * 64 + c0, r);
                            tmem_ld_wait();
#pragma unroll
                            for (int i = 0; i < 32; ++i) acc[c0 + i] += (double)__uint_as_float(r[i]);
                        }
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&s.gacc_empty[buf]);
                    }
                    g_groups += n_groups;
                    float* out = a.partials + (size_t)(t.piece % a.n_slots) * kGramElems + (size_t)row * kD + half * 64;
#pragma unroll
                    for (int i = 0; i < 64; i += 4)
                        __stcg(reinterpret_cast<float4*>(out + i),
                               make_float4((float)acc[i], (float)acc[i + 1], (float)acc[i + 2], (float)acc[i + 3]));
                    if (wtid == 0) PROF_ADD(21, tw1);
                    workers_sync();
                    if (wtid == 0) PROF_ADD(22, tw1);
                    if (wtid == 0) {
                        __threadfence();                  // releases what the other threads wrote before the barrier
                        const int done = atomicAdd(a.gram_done + t.unit, 1) + 1;
                        __threadfence();
                        if (done == unit_pieces(p, t.unit)) advance_gram_prefix(a);
                    }
                } else {
                    // ---- scoring epilogue: the two groups of four warps take alternate tiles
                    const int group = wwarp >> 2;
                    float* out = a.scores + (size_t)t.lh * p.total_tokens + t.tok_begin;
                    for (int j = 0; j < n_tiles; ++j) {
                        const int st = s_tiles + j, buf = st & 1, use = st >> 1;
                        const int og = j / kOutTiles, in_og = j % kOutTiles;
                        if (buf == group) {
                            wait(&s.sacc_full[buf], use & 1);
                            tc_fence_after_sync();
                            const uint32_t d_row = tmem + ((uint32_t)(q * 32) << 16) + kScoreCol0 + buf * 128;
                            uint32_t hi[MP / 16][16], lo[MP / 16][16];
#pragma unroll
                            for (int c = 0; c < MP / 16; ++c) {
                                tmem_ld_32x32b_x16(d_row + c * 16, hi[c]);
                                tmem_ld_32x32b_x16(d_row + MP + c * 16, lo[c]);
                            }
                            tmem_ld_wait();
                            float acc4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                            for (int c = 0; c < MP / 16; ++c)
#pragma unroll
                                for (int i = 0; i < 16; ++i) {
                                    const float v = __uint_as_float(hi[c][i]) + __uint_as_float(lo[c][i]);
                                    acc4[i & 3] = fmaf(v, v, acc4[i & 3]);
                                }
                            tc_fence_before_sync();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&s.sacc_empty[buf]);
                            s.obuf[og & 1][in_og * kTile + q * 32 + lane] = (acc4[0] + acc4[1]) + (acc4[2] + acc4[3]);
                        }
                        if (in_og == kOutTiles - 1 || j == n_tiles - 1) {
                            workers_sync();
                            const int g0 = og * kOutTiles * kTile;
                            const int count = min(t.n_tok - g0, (in_og + 1) * kTile);
                            for (int i = wtid; i < count; i += kWorkers) out[g0 + i] = s.obuf[og & 1][i];
                        }
                    }
                    s_tiles += n_tiles;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&s.tq_empty[slot]);
                if (wtid == 0) { PROF_ADD(t.type == kTaskGram ? 9 : 10, tw1); }
                continue;
            }

            // ================================================================ factor task: one row slice of one unit
            const int unit = arg, slice = arg2;
            const int lh = unit / p.batch, b = unit - lh * p.batch;
            const int n_slices = p.cu_schunks[b + 1] - p.cu_schunks[b];
            const int rows = kD / n_slices;               // rows of C in this slice: 4, 8, 16, ... 128
            const int R = rows < 8 ? rows : 8;            // rows handled at a time
            const int n_tok = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
            double* cs = s.scratch.slice.c;               // C[row0 + i][k] at [i * kLdC + k]
            for (int row0 = slice * rows; row0 < (slice + 1) * rows; row0 += 8) {
                workers_sync();                           // the previous block's products are done with cs
                if (n_tok > kExactGramTokens) {
                    const int n_part = p.cu_chunks[b + 1] - p.cu_chunks[b];
                    const int piece0 = lh * p.total_chunks + p.cu_chunks[b];
                    // A block of a partial is R x 32 float4.  Thread (sub, i, k4) adds up, in order, the partials
                    // sub, sub + nsub, ... with sixteen loads in flight (the loads are unconditional so that the
                    // compiler keeps them together); the nsub subtotals are then added in order as well.
                    const int f4_per = R * 32, nsub = kWorkers / f4_per;
                    const int sub = wtid / f4_per, idx = wtid - sub * f4_per;
                    const int i = idx >> 5, k4 = (idx & 31) * 4;
                    double acc[4] = {0.0, 0.0, 0.0, 0.0};
                    for (int pp0 = sub; pp0 < n_part; pp0 += nsub * 16) {
                        float4 v[16];
#pragma unroll
                        for (int u = 0; u < 16; ++u) {
                            const int pp = min(pp0 + u * nsub, n_part - 1);
                            v[u] = __ldcg(reinterpret_cast<const float4*>(
                                a.partials + (size_t)((piece0 + pp) % a.n_slots) * kGramElems + (size_t)(row0 + i) * kD + k4));
                        }
#pragma unroll
                        for (int u = 0; u < 16; ++u) {
                            if (pp0 + u * nsub < n_part) {
                                acc[0] += (double)v[u].x; acc[1] += (double)v[u].y;
                                acc[2] += (double)v[u].z; acc[3] += (double)v[u].w;
                            }
                        }
                    }
                    if (R < 8)
                        for (int e = wtid; e < (8 - R) * kD; e += kWorkers) cs[(R + e / kD) * kLdC + (e % kD)] = 0.0;
                    for (int turn = 0; turn < nsub; ++turn) {
                        if (sub == turn) {
                            double* dst = cs + i * kLdC + k4;
                            if (turn == 0) {
                                *reinterpret_cast<double2*>(dst) = make_double2(acc[0], acc[1]);
                                *reinterpret_cast<double2*>(dst + 2) = make_double2(acc[2], acc[3]);
                            } else {
                                double2 lo2 = *reinterpret_cast<double2*>(dst), hi2 = *reinterpret_cast<double2*>(dst + 2);
                                *reinterpret_cast<double2*>(dst) = make_double2(lo2.x + acc[0], lo2.y + acc[1]);
                                *reinterpret_cast<double2*>(dst + 2) = make_double2(hi2.x + acc[2], hi2.y + acc[3]);
                            }
                        }
                        if (turn + 1 < nsub) workers_sync();
                    }
                } else {
                    // short unit: C[rows, :] = (K^T K)[rows, :] in fp64 straight from the keys, four tokens per mma
                    const int layer = lh / p.heads, head = lh - layer * p.heads;
                    const __nv_bfloat16* kbase = a.k.ptr + layer * a.k.stride_layer + head * a.k.stride_head +
                                                 (long long)p.cu_seqlens[b] * a.k.stride_token;
                    double* keys = s.scratch.slice.keys;
                    double d[2][2] = {{0.0, 0.0}, {0.0, 0.0}};
                    constexpr int kLoads = kStageTokens * kD / kWorkers;      // 4
                    float nxt[kLoads];
                    auto fetch = [&](int t0) {
#pragma unroll
                        for (int u = 0; u < kLoads; ++u) {
                            const int e = wtid + u * kWorkers, tt = min(t0 + e / kD, n_tok - 1);
                            nxt[u] = __bfloat162float(kbase[(long long)tt * a.k.stride_token + (e % kD)]);
                            if (t0 + e / kD >= n_tok) nxt[u] = 0.f;
                        }
                    };
                    if (n_tok > 0) fetch(0);
                    for (int t0 = 0; t0 < n_tok; t0 += kStageTokens) {
                        if (t0 > 0) workers_sync();
#pragma unroll
                        for (int u = 0; u < kLoads; ++u) keys[wtid + u * kWorkers] = (double)nxt[u];
                        workers_sync();
                        if (t0 + kStageTokens < n_tok) fetch(t0 + kStageTokens);
#pragma unroll
                        for (int ks = 0; ks < kStageTokens / 4; ++ks) {
                            const double* krow = keys + (ks * 4 + fk) * kD;
                            const double bv = fr < R ? krow[row0 + fr] : 0.0;
#pragma unroll
                            for (int j = 0; j < 2; ++j) mma_f64(d[j], krow[(wwarp + 8 * j) * 8 + fr], bv);
                        }
                    }
                    // fragment (channel (wwarp + 8 j) * 8 + fr, slice rows 2 fk and 2 fk + 1)
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        cs[(2 * fk) * kLdC + (wwarp + 8 * j) * 8 + fr] = d[j][0];
                        cs[(2 * fk + 1) * kLdC + (wwarp + 8 * j) * 8 + fr] = d[j][1];
                    }
                }
                workers_sync();
                // ---- T[rows] = C[rows,:] Phi, one 8-column tile per warp, four independent chains along the contraction
                double* t_rows = a.t_buf + ((size_t)unit * kD + row0) * MP;
                for (int nt = wwarp; nt < MP / 8; nt += kWorkerWarps) {
                    double d[4][2];
#pragma unroll
                    for (int g = 0; g < 4; ++g) d[g][0] = d[g][1] = 0.0;
#pragma unroll
                    for (int k0 = 0; k0 < kD / 4; k0 += 4)
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const int k = g * (kD / 4) + k0 + fk;
                            mma_f64(d[g], cs[fr * kLdC + k], (double)s.phi[k * MP + nt * 8 + fr]);
                        }
                    if (fr < R)
                        __stcg(reinterpret_cast<double2*>(t_rows + (size_t)fr * MP + nt * 8 + 2 * fk),
                               make_double2((d[0][0] + d[1][0]) + (d[2][0] + d[3][0]), (d[0][1] + d[1][1]) + (d[2][1] + d[3][1])));
                }
            }
            workers_sync();
            if (wtid == 0) {
                PROF_ADD(11, tw1); PROF_INC(12);
                __threadfence();                          // releases what the other threads wrote before the barrier
                const int done = atomicAdd(a.slices_done + unit, 1) + 1;
                __threadfence();
                s.last = done == n_slices;
                s.flags = 0;
            }
            workers_sync();
            if (!s.last) continue;
            PROF_T(tw2);

            // ================================================================ the unit's last slice is in: G, Cholesky, W
            const int m = p.m;
            double* g = s.scratch.chol.g;                 // by columns: g[c * MP + i] = A[i][c] for i >= c
            auto wsync = [] { workers_sync(); };
            {
                // ---- G = Phi^T T, lower-triangular 8 x 8 tiles only, T staged 32 rows at a time
                const bool finite = gram_of_sketch<MP, kWorkerWarps>(a.t_buf + (size_t)unit * kD * MP, s.phi, g, s.scratch.t, wtid, wsync);
                if (!finite) atomicOr(&s.flags, COMPACTOR_STATUS_NONFINITE);
                if (wtid < MP) s.scratch.chol.inv_diag[wtid] = 0.0;
            }
            workers_sync();
            if (wtid == 0) PROF_ADD(13, tw2);
            PROF_T(tw3);
            const bool bad = (s.flags & COMPACTOR_STATUS_NONFINITE) != 0;
            if (wtid < MP) s.scratch.chol.diag0[wtid] = g[wtid * MP + wtid];
            workers_sync();
            // ---- Cholesky, right-looking by panels of eight columns: one warp factors the panel, all update what follows
            if (!bad) cholesky_panels<MP, kWorkerWarps>(g, s.scratch.chol.diag0, s.scratch.chol.inv_diag, m, wtid, &s.flags, wsync);
            workers_sync();
            if (wtid == 0) PROF_ADD(14, tw3);
            PROF_T(tw4);
            // ---- W = Phi L^-T: blocked forward substitution on fp64 mma, 16 rows of Phi per warp, then the bf16 split
            if (!bad) {
                solve_w_tiles<MP>(s.phi, g, s.scratch.chol.inv_diag, wwarp * 16, lane, a.w + (size_t)unit * w_elems_per_unit(MP));
            } else {                                      // a unit with non-finite keys gets W = 0
                __nv_bfloat16* w_unit = a.w + (size_t)unit * w_elems_per_unit(MP);
                for (int e = wtid; e < (int)w_elems_per_unit(MP); e += kWorkers) w_unit[e] = __float2bfloat16(0.f);
            }
            if (wtid == 0) PROF_ADD(20, tw4);
            workers_sync();
            if (wtid == 0) {
                asm volatile("fence.proxy.async;" ::: "memory");
                if (a.status != nullptr && s.flags != 0) atomicOr(a.status + unit, s.flags);
                st_release_u32(reinterpret_cast<unsigned*>(a.w_ready) + unit, 1u);
                __threadfence();
                advance_w_prefix(a);
                PROF_ADD(15, tw4);
                PROF_INC(16);
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
    if (threadIdx.x == 0 && s.abort && a.status != nullptr) atomicOr(a.status + last_unit, COMPACTOR_STATUS_TIMEOUT);
}

template <int MP>
cudaError_t launch_sweep_mp(const SweepArgs& a, const CUtensorMap& kmap, const CUtensorMap& wmap, int grid,
                            cudaStream_t stream) {
    const int smem = (int)sizeof(SweepSmem<MP>) + 1024;
    cudaError_t e = cudaFuncSetAttribute(sweep_kernel<MP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    sweep_kernel<MP><<<grid, kThreads, smem, stream>>>(a, kmap, wmap);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_sweep(const SweepArgs& a, int sm_count, cudaStream_t stream) {
    if (a.total_pieces == 0 || a.units == 0) return cudaSuccess;
    CUtensorMap kmap, wmap;
    if (!make_kv_tensor_map(&kmap, a.k.ptr, a.p.layers, a.p.heads, a.p.total_tokens, a.k.stride_layer, a.k.stride_head,
                            a.k.stride_token, kTile) ||
        !make_rows_tensor_map(&wmap, a.w, (long long)a.units * 2 * a.p.mp, a.p.mp))
        return cudaErrorInvalidValue;
    // one CTA per SM; never more CTAs than there is work to claim
    const long long work = (long long)a.total_pieces + a.total_ftasks;
    const int grid = (int)(work < sm_count ? work : sm_count);
    switch (a.p.mp) {
        case 16: return launch_sweep_mp<16>(a, kmap, wmap, grid, stream);
        case 32: return launch_sweep_mp<32>(a, kmap, wmap, grid, stream);
        case 48: return launch_sweep_mp<48>(a, kmap, wmap, grid, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace compactor
