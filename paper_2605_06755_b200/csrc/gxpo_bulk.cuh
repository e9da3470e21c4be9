// Bulk-copy (TMA) staging for the write-heavy sweeps (the fused probe + extrapolate sweep and
// the AdamW sweep that writes m and v back): the default for long lists, where it measures
// 2 to 4 % faster than register staging; short lists, which cannot keep one ring per SM
// busy, and the read-heavy deferred probe stay register-staged (gxpo_tune variant 2 forces
// register staging, variant 3 forces this file's kernels).
//
// One producer thread streams whole stages (one or two 2048-element tiles of every input
// array) into a shared-memory ring with cp.async.bulk (plain 1-D copies to this CTA only, from this GPU's own
// memory only); eight consumer warps pick a tile up when its mbarrier completes, do the
// same per-coordinate arithmetic as the register-staged kernel (same functions, hence the
// same bits) and store straight from registers.  All but one stage of the ring are in flight
// whatever the consumers are doing.
//
// Every wait on an mbarrier is bounded: after kWaitLimit polls the waiting thread raises
// the kernel's error word, tells the rest of the CTA to stop, and returns; the host then
// reports GXPO_ERR_TIMEOUT.  A producer that gives up first waits (bounded again) for the
// copies it already issued, so that none lands in shared memory after the CTA has gone.
#pragma once

#include "gxpo_kernels.cuh"

namespace gxpo {

constexpr int kMaxStages = 3;
constexpr int kConsumerWarps = kThreads / 32;
constexpr int kBulkThreads = kThreads + 32;         // consumers + one producer warp
constexpr unsigned kWaitLimit = 1u << 20;           // polls per wait (each poll may itself block briefly)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity) {
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// false = gave up after `limit` polls, or another thread of the CTA already did
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, unsigned parity, volatile int* stop,
                                                  unsigned limit) {
    for (unsigned i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*stop) return false;
        if (i > 1024) __nanosleep(64);
    }
    return false;
}
// global -> this CTA's shared memory; src, dst and size are multiples of 16 bytes
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, unsigned bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ FVec<8> lds_f8(const float* p) {
    FVec<8> r;
    const uint32_t a = smem_u32(p);
    // "memory": these reads must stay ahead of the arrive that hands the stage back
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(r.x[0]), "=f"(r.x[1]), "=f"(r.x[2]), "=f"(r.x[3]) : "r"(a) : "memory");
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(r.x[4]), "=f"(r.x[5]), "=f"(r.x[6]), "=f"(r.x[7]) : "r"(a + 16) : "memory");
    return r;
}
__device__ __forceinline__ FVec<8> lds_g8(const float* p) { return lds_f8(p); }
__device__ __forceinline__ FVec<8> lds_g8(const uint16_t* p) {
    HVec<8> h;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(h.x[0]), "=r"(h.x[1]), "=r"(h.x[2]), "=r"(h.x[3]) : "r"(smem_u32(p)) : "memory");
    FVec<8> r;
#pragma unroll
    for (int i = 0; i < 4; ++i) { r.x[2 * i] = bf16_lo(h.x[i]); r.x[2 * i + 1] = bf16_hi(h.x[i]); }
    return r;
}

// one chunk of one tensor, pointers resolved
template <typename G> struct FusedUnit {
    const float* t1; const float* t0; float* out; float* m; float* v; const G* g0; const G* g1;
    uint16_t* wb;
    int len, full_tiles;                // full_tiles > 0 only when every pointer is 32-byte aligned
    bool vec;
};

// Work unit u = piece `u mod 2^unit_shift` of chunk `u >> unit_shift` (whole, half or quarter chunks:
// always a whole number of stages).  Short lists are dealt in smaller units so that the last
// round of the round-robin leaves few CTAs idle.
template <bool ADAMW, typename G, bool DEFER>
__device__ __forceinline__ bool fused_resolve(long long u, int unit_shift, const TensorDesc* descs, const ChunkRef* chunks,
                                              const TensorDesc& flat, const FusedParams& p, int stage_elems,
                                              FusedUnit<G>& U) {
    const long long c = u >> unit_shift;
    const int unit_len = kChunk >> unit_shift;
    ChunkRef ref;
    TensorDesc d;
    if (chunks) { ref = chunks[c]; d = descs[ref.tensor]; }
    else { ref.tensor = 0; ref.chunk = (unsigned)c; d = flat; }
    const long long off = (long long)ref.chunk * kChunk + (long long)(u & ((1 << unit_shift) - 1)) * unit_len;
    const long long rem = d.n - off;
    U.len = 0; U.full_tiles = 0; U.vec = false;
    if (rem <= 0) return false;
    U.len = rem < unit_len ? (int)rem : unit_len;
    U.t1 = (p.step.in_sel ? d.work : d.theta) + off;
    U.t0 = (p.ex.theta0_sel ? d.work : d.theta) + off;
    U.out = d.theta + off;
    U.m = ADAMW ? d.m + off : nullptr;
    U.v = ADAMW ? d.v + off : nullptr;
    U.g0 = reinterpret_cast<const G*>(d.g[0]) + off;
    U.g1 = reinterpret_cast<const G*>(d.g[1]) + off;
    U.wb = d.wb ? d.wb + off : nullptr;
    U.vec = (DEFER || aligned32(U.t1)) && aligned32(U.t0) && aligned32(U.out) && aligned32(U.g0) &&
            aligned32(U.g1) && (!ADAMW || (aligned32(U.m) && aligned32(U.v))) && aligned16(U.wb);
    U.full_tiles = U.vec ? U.len / stage_elems : 0;
    return true;
}

// sum over the 256 consumer threads on named barrier 1 (the producer warp takes no part);
// valid in thread 0
__device__ __forceinline__ double consumer_sum(double x, double* smem8) {
    x = warp_sum(x);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("bar.sync 1, %0;" :: "r"(kThreads) : "memory");
    if (lane == 0) smem8[warp] = x;
    asm volatile("bar.sync 1, %0;" :: "r"(kThreads) : "memory");
    double t = 0.0;
    if (warp == 0) { t = (lane < kConsumerWarps) ? smem8[lane] : 0.0; t = warp_sum(t); }
    return t;
}
// Shared memory per stage: [theta1 unless DEFER] theta0 [m v if ADAMW] g0 g1, kMult tiles each.
// Ring shape, measured on a 7.6e9-parameter list: what matters is about 64 KB in flight per SM
// in as few, as large pieces as possible.  Deferred sweep (5 arrays): 2 stages of 4096
// elements 6.62 TB/s, 3 of 2048 6.53, 2 of 2048 5.77, 4 of 2048 6.10, 3 of 4096 6.09.  The
// non-deferred sweep (6 arrays) does best with 3 stages of 2048.
// LIGHT (deferred AdamW sweep that leaves m and v unwritten: 16 R + 4 W) is bound by
// latency rather than by the write path: two CTAs per SM, each with 3 stages of 2048
// (23.5 ms on a 7.6e9-parameter list; 2 stages 23.65).
template <bool ADAMW, typename G, bool DEFER, bool LIGHT = false>
struct BulkLayout {
    static constexpr int kMult = (DEFER && !LIGHT) ? 2 : 1;      // tiles per stage
    static constexpr int kStagesN = (DEFER && !LIGHT) ? 2 : 3;
    static constexpr int kElems = kTile * kMult;
    static constexpr unsigned kF = kElems * sizeof(float);
    static constexpr unsigned kGb = kElems * sizeof(G);
    static constexpr unsigned kStage = ((DEFER ? 1 : 2) + (ADAMW ? 2 : 0)) * kF + 2 * kGb;
    static constexpr unsigned kTotal = kStagesN * kStage + 2 * kMaxStages * sizeof(uint64_t) + 16;
};

template <bool ADAMW, typename G, bool DEFER, bool DIAG, bool LIGHT>
__device__ __forceinline__ void fused_bulk_body(const TensorDesc* __restrict__ descs, const ChunkRef* __restrict__ chunks,
                                                long long num_chunks, const TensorDesc& flat, const FusedParams& p,
                                                int unit_shift, int* error_word, double* diag_partials,
                                                unsigned* ticket, double* diag_out) {
    typedef BulkLayout<ADAMW, G, DEFER, LIGHT> L;
    const long long num_units = num_chunks << unit_shift;
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int kStages = L::kStagesN;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStages * L::kStage);
    uint64_t* empty = full + kMaxStages;
    volatile int* stop = reinterpret_cast<volatile int*>(empty + kMaxStages);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, kConsumerWarps); }
        *stop = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (warp == kConsumerWarps) {                       // ---- producer warp: lane 0 issues the copies
        if (lane != 0) return;
        unsigned it = 0;
        bool ok = true;
        for (long long u = blockIdx.x; u < num_units && ok; u += gridDim.x) {
            FusedUnit<G> U;
            if (!fused_resolve<ADAMW, G, DEFER>(u, unit_shift, descs, chunks, flat, p, L::kElems, U)) continue;
            for (int j = 0; j < U.full_tiles; ++j, ++it) {
                const unsigned s = it % kStages, n = it / kStages;
                // the consumers must have released the stage's previous use
                if (n > 0 && !mbar_wait_bounded(empty + s, (n - 1) & 1, stop, kWaitLimit)) { ok = false; break; }
                unsigned char* st = smem + s * L::kStage;
                const int e = j * L::kElems;
                mbar_expect_tx(full + s, L::kStage);
                unsigned o = 0;
                if (!DEFER) { bulk_load(st, U.t1 + e, L::kF, full + s); o += L::kF; }
                bulk_load(st + o, U.t0 + e, L::kF, full + s); o += L::kF;
                if (ADAMW) {
                    bulk_load(st + o, U.m + e, L::kF, full + s); o += L::kF;
                    bulk_load(st + o, U.v + e, L::kF, full + s); o += L::kF;
                }
                bulk_load(st + o, U.g0 + e, L::kGb, full + s); o += L::kGb;
                bulk_load(st + o, U.g1 + e, L::kGb, full + s);
            }
        }
        if (!ok) {
            *stop = 1;
            atomicExch(error_word, 1);
            // copies already issued still target this CTA's shared memory: give each of the
            // last kStages uses a bounded chance to land before the CTA goes away
            for (unsigned k = 0; k < (unsigned)kStages && k < it; ++k) {
                const unsigned i2 = it - 1 - k;
                for (unsigned w = 0; w < kWaitLimit && !mbar_try_wait(full + i2 % kStages, (i2 / kStages) & 1); ++w)
                    __nanosleep(64);
            }
        }
        return;
    }

    // ---- consumers
    __shared__ double red[8];
    __shared__ bool is_last;
    DiagAcc acc;
    if (DIAG) {
#pragma unroll
        for (int q = 0; q < kDiagN; ++q) acc.v[q] = 0.0;
    }
    bool alive = true;
    const float gs0 = p.ex.gscale0 ? __ldg(p.ex.gscale0) : 1.0f, gs1 = p.ex.gscale1 ? __ldg(p.ex.gscale1) : 1.0f;
    unsigned it = 0;
    for (long long u = blockIdx.x; u < num_units && alive; u += gridDim.x) {
        FusedUnit<G> U;
        if (!fused_resolve<ADAMW, G, DEFER>(u, unit_shift, descs, chunks, flat, p, L::kElems, U)) continue;
        if (!U.vec) {                                   // misaligned tensor: scalar path, no staging
            for (int e = threadIdx.x; e < U.len; e += kThreads) {
                float mm = ADAMW ? U.m[e] : 0.0f, vv = ADAMW ? U.v[e] : 0.0f;
                const float x = fused_elem<ADAMW, DEFER, DIAG>(DEFER ? 0.0f : U.t1[e], U.t0[e], mm, vv,
                                                                __fmul_rn(ld_grad1(U.g0 + e), gs0),
                                                                __fmul_rn(ld_grad1(U.g1 + e), gs1), p, &acc);
                if (!p.step.skip_out) U.out[e] = x;
                if (U.wb) U.wb[e] = to_bf16(x);
                if (ADAMW && !LIGHT && p.step.write_state) { U.m[e] = mm; U.v[e] = vv; }
            }
            continue;
        }
        for (int j = 0; j < U.full_tiles; ++j, ++it) {
            const unsigned s = it % kStages, n = it / kStages;
            if (!mbar_wait_bounded(full + s, n & 1, stop, kWaitLimit)) {
                *stop = 1;
                atomicExch(error_word, 1);
                alive = false;
                break;
            }
            const unsigned char* st = smem + s * L::kStage;
#pragma unroll 1
            for (int h = 0; h < L::kMult; ++h) {
            const int tt = (h * kThreads + threadIdx.x) * 8;
            unsigned o = 0;
            FVec<8> a1, a0, mm, vv;
            if (!DEFER) { a1 = lds_f8(reinterpret_cast<const float*>(st) + tt); o += L::kF; }
            a0 = lds_f8(reinterpret_cast<const float*>(st + o) + tt); o += L::kF;
            if (ADAMW) {
                mm = lds_f8(reinterpret_cast<const float*>(st + o) + tt); o += L::kF;
                vv = lds_f8(reinterpret_cast<const float*>(st + o) + tt); o += L::kF;
            }
            FVec<8> b0 = scaled<8>(lds_g8(reinterpret_cast<const G*>(st + o) + tt), gs0); o += L::kGb;
            FVec<8> b1 = scaled<8>(lds_g8(reinterpret_cast<const G*>(st + o) + tt), gs1);
            const int e = j * L::kElems + tt;
            if (DEFER) {
                a1 = a0;
                optim_step_vec<ADAMW, 8>(a1, mm, vv, b0, p.step0);
            }
            optim_step_vec<ADAMW, 8>(a1, mm, vv, b1, p.step);
            extrapolate_vec<8, DIAG>(a1, a0, b0, b1, p.ex, &acc);
            if (!p.step.skip_out) st_f(U.out + e, a1);
            if (U.wb) st_bf16(U.wb + e, a1);
            if (ADAMW && !LIGHT && p.step.write_state) { st_f(U.m + e, mm); st_f(U.v + e, vv); }
            }
            // Hand the stage back only now: every lane's stores depend on what it read from
            // the stage, so by this point the shared-memory reads have certainly completed.
            __syncwarp();
            if (lane == 0) mbar_arrive(empty + s);
        }
        if (!alive) break;
        // ragged rest of the chunk (less than one stage): register path
        const int done = U.full_tiles * L::kElems;
        if (done < U.len)
            fused_chunk_vec<ADAMW, G, 8, DEFER, DIAG>(U.out + done, U.t1 + done, U.t0 + done,
                                                       ADAMW ? U.m + done : nullptr, ADAMW ? U.v + done : nullptr,
                                                       U.g0 + done, U.g1 + done, U.len - done, p, gs0, gs1, &acc,
                                                       U.wb ? U.wb + done : nullptr);
    }
    if (DIAG) {
        // every consumer thread gets here, also after a wait that gave up
#pragma unroll
        for (int q = 0; q < kDiagN; ++q) {
            const double tot = consumer_sum(acc.v[q], red);
            if (threadIdx.x == 0) diag_partials[q * kMaxGrid + blockIdx.x] = tot;
        }
        if (threadIdx.x == 0) {
            __threadfence();
            is_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
        }
        asm volatile("bar.sync 1, %0;" :: "r"(kThreads) : "memory");
        if (is_last) {
            __threadfence();
#pragma unroll 1
            for (int q = 0; q < kDiagN; ++q) {
                double sum = 0.0;
                for (unsigned i = threadIdx.x; i < gridDim.x; i += kThreads) sum += __ldcg(diag_partials + q * kMaxGrid + i);
                sum = consumer_sum(sum, red);
                if (threadIdx.x == 0) diag_out[q] = sum;
            }
            if (threadIdx.x == 0) *ticket = 0u;
        }
    }
}

template <bool ADAMW, typename G, bool DEFER, bool DIAG>
__global__ void __launch_bounds__(kBulkThreads, 1)
fused_bulk_kernel(const TensorDesc* __restrict__ descs, const ChunkRef* __restrict__ chunks,
                  long long num_chunks, TensorDesc flat, FusedParams p, int unit_shift, int* error_word,
                  double* diag_partials, unsigned* ticket, double* diag_out) {
    fused_bulk_body<ADAMW, G, DEFER, DIAG, false>(descs, chunks, num_chunks, flat, p, unit_shift, error_word, diag_partials, ticket, diag_out);
}

// The LIGHT shape, two CTAs per SM: 18 warps put 5 on one scheduler, whose 16384 registers
// then allow 96 per thread (the compiler spills 76 bytes; measured 23.7 ms against 24.6 with
// one CTA and against 29.2 ms at 112 registers, where only one CTA fits).
template <typename G>
__global__ void __launch_bounds__(kBulkThreads, 2)
fused_bulk_light_kernel(const TensorDesc* __restrict__ descs, const ChunkRef* __restrict__ chunks,
                        long long num_chunks, TensorDesc flat, FusedParams p, int unit_shift, int* error_word,
                        double* diag_partials, unsigned* ticket, double* diag_out) {
    fused_bulk_body<true, G, true, false, true>(descs, chunks, num_chunks, flat, p, unit_shift, error_word, diag_partials, ticket, diag_out);
}

// ---------------------------------------------------------------------------
// The AdamW sweep with the same staging, for the calls that write m and v back (slow
// step, fallback step, non-deferred probe steps): 14 R + 12 W per parameter.  Measured on a
// 7.6e9-parameter list: two stages of 4096 elements 6.55 TB/s against 6.43 register-staged
// (three stages of 2048: 6.34; two of 8192: 6.04).  The read-heavy deferred probe (14 R +
// 4 W) is slower staged (5.8 against 6.8 TB/s) and stays register-staged.  Consumers
// accumulate sum(g^2) like the register-staged kernel and reduce it among themselves on a
// named barrier (the producer warp has left by then).
// MODE bit kStepDot: the sweep also stages g0 and accumulates <g0, g> for the diagnostics'
// cosine (+2 bytes per parameter for bfloat16 gradients instead of a separate 4-byte pass);
// products are summed like dot_kernel's.
// MODE bit kStepReplay: m and v are still those from before the two probe steps (the fused
// sweep left them unwritten as well); g0 and g1 are staged too and both moment updates are
// replayed in registers before the step itself: 18 R + 12 W, and the fused sweep before it
// saves its 8 bytes of state writes.
// ---------------------------------------------------------------------------
constexpr int kStepDot = 1, kStepReplay = 2;
constexpr int kStepMult = 2;       // tiles per stage
constexpr int kStepStages = 2;
template <bool ADAMW, typename G, int MODE>
struct StepLayout {
    static constexpr int kElems = kTile * kStepMult;
    static constexpr unsigned kF = kElems * sizeof(float);
    static constexpr unsigned kGb = kElems * sizeof(G);
    static constexpr int kGrads = 1 + (MODE != 0 ? 1 : 0) + ((MODE & kStepReplay) ? 1 : 0);   // g [g0 [g1]]
    static constexpr unsigned kStage = (ADAMW ? 3 : 1) * kF + kGrads * kGb;
    static constexpr unsigned kTotal = kStepStages * kStage + 2 * kMaxStages * sizeof(uint64_t) + 16;
};
template <typename G> struct StepUnit {
    const float* in; float* out; float* snap; float* m; float* v; const G* g; const G* g0; const G* g1; uint16_t* wb;
    int len, full_tiles; bool vec;
};
template <bool ADAMW, typename G, int MODE>
__device__ __forceinline__ bool step_resolve(long long u, int unit_shift, const TensorDesc* descs, const ChunkRef* chunks,
                                             const TensorDesc& flat, const StepParams& p, int stage_elems, StepUnit<G>& U) {
    const long long c = u >> unit_shift;
    const int unit_len = kChunk >> unit_shift;
    ChunkRef ref; TensorDesc d;
    if (chunks) { ref = chunks[c]; d = descs[ref.tensor]; } else { ref.tensor = 0; ref.chunk = (unsigned)c; d = flat; }
    const long long off = (long long)ref.chunk * kChunk + (long long)(u & ((1 << unit_shift) - 1)) * unit_len;
    const long long rem = d.n - off;
    U.len = 0; U.full_tiles = 0; U.vec = false;
    if (rem <= 0) return false;
    U.len = rem < unit_len ? (int)rem : unit_len;
    U.in = (p.in_sel ? d.work : d.theta) + off;
    U.out = (p.out_sel ? d.work : d.theta) + off;
    U.snap = p.snapshot ? d.work + off : nullptr;
    U.m = ADAMW ? d.m + off : nullptr; U.v = ADAMW ? d.v + off : nullptr;
    const void* gsel = p.which_grad == 0 ? d.g[0] : (p.which_grad == 1 ? d.g[1] : d.g[2]);
    U.g = reinterpret_cast<const G*>(gsel) + off;
    U.g0 = MODE ? reinterpret_cast<const G*>(d.g[0]) + off : nullptr;
    U.g1 = (MODE & kStepReplay) ? reinterpret_cast<const G*>(d.g[1]) + off : nullptr;
    U.wb = (p.emit && d.wb) ? d.wb + off : nullptr;
    U.vec = aligned32(U.in) && aligned32(U.out) && aligned32(U.g) && (!ADAMW || (aligned32(U.m) && aligned32(U.v))) &&
            (!p.snapshot || aligned32(U.snap)) && aligned16(U.wb) && aligned32(U.g0) && aligned32(U.g1);   // null passes
    U.full_tiles = U.vec ? U.len / stage_elems : 0;
    return true;
}
// <a, b> over [0, len) by the 256 consumer threads, added to acc (the short pieces that
// bypass the ring)
template <typename G>
__device__ __forceinline__ void consumer_dot(const G* a, const G* b, int len, double& acc) {
    for (int e = threadIdx.x; e < len; e += kThreads) acc += (double)ld_grad1(a + e) * (double)ld_grad1(b + e);
}

// The pieces that bypass the ring, replay mode: advance m and v in place with g0 and g1, after
// which the ordinary code paths apply.  Every thread advances exactly the elements it will
// read back itself (VEC: the vectors and the tail element step_chunk_vec<.., 8> gives it;
// otherwise step_chunk_scalar's stride), so no barrier is needed, only program order.
template <typename G, bool VEC>
__device__ __forceinline__ void consumer_replay(float* m, float* v, const G* g0, const G* g1, int len,
                                                const StepParams& p, float gs0, float gs1) {
    auto one = [&](int e) {
        float mm = m[e], vv = v[e];
        advance_moments_elem(mm, vv, __fmul_rn(ld_grad1(g0 + e), gs0), p);
        advance_moments_elem(mm, vv, __fmul_rn(ld_grad1(g1 + e), gs1), p);
        m[e] = mm; v[e] = vv;
    };
    if (VEC) {
        const int nvec = len / 8;
        for (int iv = threadIdx.x; iv < nvec; iv += kThreads)
            for (int i = 0; i < 8; ++i) one(iv * 8 + i);
        const int e = nvec * 8 + threadIdx.x;
        if (e < len) one(e);
    } else {
        for (int e = threadIdx.x; e < len; e += kThreads) one(e);
    }
    asm volatile("" ::: "memory");          // the loads that follow are asm statements
}

template <bool ADAMW, typename G, int MODE>
__global__ void __launch_bounds__(kBulkThreads, 1)
step_bulk_kernel(const TensorDesc* __restrict__ descs, const ChunkRef* __restrict__ chunks,
                 long long num_chunks, TensorDesc flat, StepParams p, int unit_shift, double* partials, unsigned* ticket,
                 double* sumsq_out, int* error_word, double* dot_partials, double* dot_out) {
    typedef StepLayout<ADAMW, G, MODE> L;
    const long long num_units = num_chunks << unit_shift;
    constexpr bool DOT = (MODE & kStepDot) != 0, REPLAY = (MODE & kStepReplay) != 0;
    constexpr int kStages = kStepStages;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ double red[8];
    __shared__ bool is_last;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStages * L::kStage);
    uint64_t* empty = full + kMaxStages;
    volatile int* stop = reinterpret_cast<volatile int*>(empty + kMaxStages);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, kConsumerWarps); }
        *stop = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == kConsumerWarps) {
        if (lane != 0) return;
        unsigned it = 0; bool ok = true;
        for (long long u = blockIdx.x; u < num_units && ok; u += gridDim.x) {
            StepUnit<G> U;
            if (!step_resolve<ADAMW, G, MODE>(u, unit_shift, descs, chunks, flat, p, L::kElems, U)) continue;
            for (int j = 0; j < U.full_tiles; ++j, ++it) {
                const unsigned s = it % kStages, n = it / kStages;
                if (n > 0 && !mbar_wait_bounded(empty + s, (n - 1) & 1, stop, kWaitLimit)) { ok = false; break; }
                unsigned char* st = smem + s * L::kStage;
                const int e = j * L::kElems;
                mbar_expect_tx(full + s, L::kStage);
                unsigned o = 0;
                bulk_load(st, U.in + e, L::kF, full + s); o += L::kF;
                if (ADAMW) { bulk_load(st + o, U.m + e, L::kF, full + s); o += L::kF; bulk_load(st + o, U.v + e, L::kF, full + s); o += L::kF; }
                bulk_load(st + o, U.g + e, L::kGb, full + s); o += L::kGb;
                if (MODE) { bulk_load(st + o, U.g0 + e, L::kGb, full + s); o += L::kGb; }
                if (REPLAY) bulk_load(st + o, U.g1 + e, L::kGb, full + s);
            }
        }
        if (!ok) {
            *stop = 1; atomicExch(error_word, 1);
            for (unsigned k = 0; k < (unsigned)kStages && k < it; ++k) {
                const unsigned i2 = it - 1 - k;
                for (unsigned w = 0; w < kWaitLimit && !mbar_try_wait(full + i2 % kStages, (i2 / kStages) & 1); ++w) __nanosleep(64);
            }
        }
        return;
    }
    const float gscale = p.gscale ? __ldg(p.gscale) : 1.0f;
    const float gs0 = (REPLAY && p.gscale_r0) ? __ldg(p.gscale_r0) : 1.0f;
    const float gs1 = (REPLAY && p.gscale_r1) ? __ldg(p.gscale_r1) : 1.0f;
    double acc = 0.0, accd = 0.0; unsigned it = 0; bool alive = true;
    for (long long u = blockIdx.x; u < num_units && alive; u += gridDim.x) {
        StepUnit<G> U;
        if (!step_resolve<ADAMW, G, MODE>(u, unit_shift, descs, chunks, flat, p, L::kElems, U)) continue;
        if (!U.vec) {
            if (REPLAY) consumer_replay<G, false>(U.m, U.v, U.g0, U.g1, U.len, p, gs0, gs1);
            step_chunk_scalar<ADAMW, G>(U.out, U.in, U.snap, U.m, U.v, U.g, U.len, p, gscale, acc, U.wb);
            if (DOT) consumer_dot(U.g0, U.g, U.len, accd);
            continue;
        }
        for (int j = 0; j < U.full_tiles; ++j, ++it) {
            const unsigned s = it % kStages, n = it / kStages;
            if (!mbar_wait_bounded(full + s, n & 1, stop, kWaitLimit)) { *stop = 1; atomicExch(error_word, 1); alive = false; break; }
            const unsigned char* st = smem + s * L::kStage;
#pragma unroll 1
            for (int h = 0; h < kStepMult; ++h) {
                const int tt = (h * kThreads + threadIdx.x) * 8;
                unsigned o = 0;
                FVec<8> th, mm, vv;
                th = lds_f8(reinterpret_cast<const float*>(st) + tt); o += L::kF;
                if (ADAMW) { mm = lds_f8(reinterpret_cast<const float*>(st + o) + tt); o += L::kF; vv = lds_f8(reinterpret_cast<const float*>(st + o) + tt); o += L::kF; }
                const FVec<8> gg = lds_g8(reinterpret_cast<const G*>(st + o) + tt); o += L::kGb;
                if (MODE) {
                    const FVec<8> g0 = lds_g8(reinterpret_cast<const G*>(st + o) + tt); o += L::kGb;
                    if (DOT) {
                        float dq = 0.0f;
#pragma unroll
                        for (int i = 0; i < 8; ++i) dq = fmaf(g0.x[i], gg.x[i], dq);
                        accd += (double)dq;
                    }
                    if (REPLAY) {
                        const FVec<8> g1 = lds_g8(reinterpret_cast<const G*>(st + o) + tt);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            advance_moments_elem(mm.x[i], vv.x[i], __fmul_rn(g0.x[i], gs0), p);
                            advance_moments_elem(mm.x[i], vv.x[i], __fmul_rn(g1.x[i], gs1), p);
                        }
                    }
                }
                const int e = j * L::kElems + tt;
                if (U.snap) st_f(U.snap + e, th);
                float sq = 0.0f;
#pragma unroll
                for (int i = 0; i < 8; ++i) { sq = fmaf(gg.x[i], gg.x[i], sq); optim_step_elem<ADAMW>(th.x[i], mm.x[i], vv.x[i], __fmul_rn(gg.x[i], gscale), p); }
                if (!p.skip_out) st_f(U.out + e, th);
                if (U.wb) st_bf16(U.wb + e, th);
                if (ADAMW && p.write_state) { st_f(U.m + e, mm); st_f(U.v + e, vv); }
                acc += (double)sq;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty + s);
        }
        if (!alive) break;
        const int done = U.full_tiles * L::kElems;
        if (done < U.len) {
            if (REPLAY) consumer_replay<G, true>(U.m + done, U.v + done, U.g0 + done, U.g1 + done, U.len - done, p, gs0, gs1);
            step_chunk_vec<ADAMW, G, 8>(U.out + done, U.in + done, U.snap ? U.snap + done : nullptr, ADAMW ? U.m + done : nullptr,
                                        ADAMW ? U.v + done : nullptr, U.g + done, U.len - done, p, gscale, acc, U.wb ? U.wb + done : nullptr);
            if (DOT) consumer_dot(U.g0 + done, U.g + done, U.len - done, accd);
        }
    }
    if (p.want_norm) {                                   // DOT comes only with want_norm
        const double tot = consumer_sum(acc, red);
        double totd = 0.0;
        if (DOT) totd = consumer_sum(accd, red);
        if (threadIdx.x == 0) {
            partials[blockIdx.x] = tot;
            if (DOT) dot_partials[blockIdx.x] = totd;
            __threadfence();
            is_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
        }
        asm volatile("bar.sync 1, %0;" :: "r"(kThreads) : "memory");
        if (is_last) {
            __threadfence();
            double sum = 0.0, sumd = 0.0;
            for (unsigned i = threadIdx.x; i < gridDim.x; i += kThreads) {
                sum += __ldcg(partials + i);
                if (DOT) sumd += __ldcg(dot_partials + i);
            }
            sum = consumer_sum(sum, red);
            if (DOT) sumd = consumer_sum(sumd, red);
            if (threadIdx.x == 0) {
                *sumsq_out = sum;
                if (DOT) *dot_out = sumd;
                *ticket = 0u;
            }
        }
    }
}

// ---------------------------------------------------------------------------
// The slow step for trainers whose model runs on the bfloat16 copies only: the fused sweep
// stored theta-tilde as bfloat16 and nothing else (theta^t is still in `theta`, m and v still
// predate the probe steps), so this sweep stages theta^t, m, v, g_slow, g0 and g1 -- the very
// arrays of the replaying sweep -- redoes both probe steps and the extrapolation in registers
// with the functions of the fused sweep (hence the same float32 theta-tilde, bit for bit, whose
// rounding the caller's third backward pass saw), and takes the slow step from there:
// 18 R + 12 W (+2 for the bfloat16 copy of theta^{t+1}), and no float32 theta-tilde or
// theta^{t,1} ever reaches memory.
// ---------------------------------------------------------------------------
// SHAPE 0: one CTA per SM, two stages of 4096 elements (the replaying sweep's ring).
// SHAPE 1: two CTAs per SM, three stages of 2048 elements each (the light fused sweep's ring):
// this sweep carries the arithmetic of both, and eight consumer warps per SM cannot hide it.
template <typename G, int SHAPE>
struct RecomputeLayout {
    static constexpr int kMult = SHAPE ? 1 : 2;
    static constexpr int kStagesN = SHAPE ? 3 : 2;
    static constexpr int kElems = kTile * kMult;
    static constexpr unsigned kF = kElems * sizeof(float);
    static constexpr unsigned kGb = kElems * sizeof(G);
    static constexpr unsigned kStage = 3 * kF + 3 * kGb;       // theta^t, m, v, g_slow, g0, g1
    static constexpr unsigned kTotal = kStagesN * kStage + 2 * kMaxStages * sizeof(uint64_t) + 16;
};
template <typename G, int SHAPE>
__global__ void __launch_bounds__(kBulkThreads, SHAPE ? 2 : 1)
slow_recompute_bulk_kernel(const TensorDesc* __restrict__ descs, const ChunkRef* __restrict__ chunks,
                           long long num_chunks, TensorDesc flat, FusedParams fp, StepParams p, int unit_shift,
                           double* partials, unsigned* ticket, double* sumsq_out, int* error_word) {
    typedef RecomputeLayout<G, SHAPE> L;
    constexpr int kStages = L::kStagesN;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ double red[8];
    __shared__ bool is_last;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStages * L::kStage);
    uint64_t* empty = full + kMaxStages;
    volatile int* stop = reinterpret_cast<volatile int*>(empty + kMaxStages);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, kConsumerWarps); }
        *stop = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const long long num_units = num_chunks << unit_shift;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == kConsumerWarps) {                       // ---- producer: same stage layout as the replaying sweep
        if (lane != 0) return;
        unsigned it = 0; bool ok = true;
        for (long long u = blockIdx.x; u < num_units && ok; u += gridDim.x) {
            StepUnit<G> U;
            if (!step_resolve<true, G, kStepReplay>(u, unit_shift, descs, chunks, flat, p, L::kElems, U)) continue;
            for (int j = 0; j < U.full_tiles; ++j, ++it) {
                const unsigned s = it % kStages, n = it / kStages;
                if (n > 0 && !mbar_wait_bounded(empty + s, (n - 1) & 1, stop, kWaitLimit)) { ok = false; break; }
                unsigned char* st = smem + s * L::kStage;
                const int e = j * L::kElems;
                mbar_expect_tx(full + s, L::kStage);
                unsigned o = 0;
                bulk_load(st, U.in + e, L::kF, full + s); o += L::kF;
                bulk_load(st + o, U.m + e, L::kF, full + s); o += L::kF;
                bulk_load(st + o, U.v + e, L::kF, full + s); o += L::kF;
                bulk_load(st + o, U.g + e, L::kGb, full + s); o += L::kGb;
                bulk_load(st + o, U.g0 + e, L::kGb, full + s); o += L::kGb;
                bulk_load(st + o, U.g1 + e, L::kGb, full + s);
            }
        }
        if (!ok) {
            *stop = 1; atomicExch(error_word, 1);
            for (unsigned k = 0; k < (unsigned)kStages && k < it; ++k) {
                const unsigned i2 = it - 1 - k;
                for (unsigned w = 0; w < kWaitLimit && !mbar_try_wait(full + i2 % kStages, (i2 / kStages) & 1); ++w) __nanosleep(64);
            }
        }
        return;
    }
    const float gscale = p.gscale ? __ldg(p.gscale) : 1.0f;
    const float gs0 = fp.ex.gscale0 ? __ldg(fp.ex.gscale0) : 1.0f, gs1 = fp.ex.gscale1 ? __ldg(fp.ex.gscale1) : 1.0f;
    double acc = 0.0; unsigned it = 0; bool alive = true;
    for (long long u = blockIdx.x; u < num_units && alive; u += gridDim.x) {
        StepUnit<G> U;
        if (!step_resolve<true, G, kStepReplay>(u, unit_shift, descs, chunks, flat, p, L::kElems, U)) continue;
        for (int j = 0; j < U.full_tiles; ++j, ++it) {
            const unsigned s = it % kStages, n = it / kStages;
            if (!mbar_wait_bounded(full + s, n & 1, stop, kWaitLimit)) { *stop = 1; atomicExch(error_word, 1); alive = false; break; }
            const unsigned char* st = smem + s * L::kStage;
#pragma unroll 1
            for (int h = 0; h < L::kMult; ++h) {
                const int tt = (h * kThreads + threadIdx.x) * 8;
                unsigned o = 0;
                const FVec<8> th0 = lds_f8(reinterpret_cast<const float*>(st) + tt); o += L::kF;
                FVec<8> mm = lds_f8(reinterpret_cast<const float*>(st + o) + tt); o += L::kF;
                FVec<8> vv = lds_f8(reinterpret_cast<const float*>(st + o) + tt); o += L::kF;
                const FVec<8> gg = lds_g8(reinterpret_cast<const G*>(st + o) + tt); o += L::kGb;
                const FVec<8> b0 = scaled<8>(lds_g8(reinterpret_cast<const G*>(st + o) + tt), gs0); o += L::kGb;
                const FVec<8> b1 = scaled<8>(lds_g8(reinterpret_cast<const G*>(st + o) + tt), gs1);
                FVec<8> th = th0;
                optim_step_vec<true, 8>(th, mm, vv, b0, fp.step0);
                optim_step_vec<true, 8>(th, mm, vv, b1, fp.step);
                extrapolate_vec<8, false>(th, th0, b0, b1, fp.ex, nullptr);          // th = theta-tilde
                float sq = 0.0f;
#pragma unroll
                for (int i = 0; i < 8; ++i) sq = fmaf(gg.x[i], gg.x[i], sq);
                optim_step_vec<true, 8>(th, mm, vv, scaled<8>(gg, gscale), p);      // same roundings as optim_step_elem
                const int e = j * L::kElems + tt;
                st_f(U.out + e, th);
                if (U.wb) st_bf16(U.wb + e, th);
                st_f(U.m + e, mm); st_f(U.v + e, vv);
                acc += (double)sq;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty + s);
        }
        if (!alive) break;
        // what bypasses the ring (ragged ends, misaligned tensors): coordinate by coordinate
        for (int e = U.full_tiles * L::kElems + threadIdx.x; e < U.len; e += kThreads) {
            float mm = U.m[e], vv = U.v[e];
            const float gg = ld_grad1(U.g + e);
            float x = fused_elem<true, true, false>(0.0f, U.in[e], mm, vv, __fmul_rn(ld_grad1(U.g0 + e), gs0),
                                                    __fmul_rn(ld_grad1(U.g1 + e), gs1), fp, nullptr);
            optim_step_elem<true>(x, mm, vv, __fmul_rn(gg, gscale), p);
            U.out[e] = x;
            if (U.wb) U.wb[e] = to_bf16(x);
            U.m[e] = mm; U.v[e] = vv;
            acc += (double)(gg * gg);
        }
    }
    const double tot = consumer_sum(acc, red);
    if (threadIdx.x == 0) {
        partials[blockIdx.x] = tot;
        __threadfence();
        is_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    }
    asm volatile("bar.sync 1, %0;" :: "r"(kThreads) : "memory");
    if (is_last) {
        __threadfence();
        double sum = 0.0;
        for (unsigned i = threadIdx.x; i < gridDim.x; i += kThreads) sum += __ldcg(partials + i);
        sum = consumer_sum(sum, red);
        if (threadIdx.x == 0) { *sumsq_out = sum; *ticket = 0u; }
    }
}

// Nothing ever completes the barrier this kernel waits on: the bounded wait has to give up
// after `limit` polls and raise the error word.  Used to check that path end to end.
__global__ void bounded_wait_probe_kernel(unsigned limit, int* error_word) {
    __shared__ uint64_t bar;
    __shared__ int stop_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        stop_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait_bounded(&bar, 0, &stop_flag, limit)) atomicExch(error_word, 1);
    }
}

}  // namespace gxpo
