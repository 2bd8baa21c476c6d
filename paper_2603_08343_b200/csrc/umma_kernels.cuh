// tcgen05 kernel family for bf16 rows, d = 1024 * PIECES (1024 ... 8192), many rows.
//
// H_d = H_2 (x) ... (x) H_2 acts on the index bits independently, so the seven
// stages on index bits 3..9 are one product with H_128.  A row piece of 1024
// contiguous bf16 elements is, as it lies in memory, a 128 x 8 matrix
// B[k][n] = x[k*8 + n]   (k = bits 3..9, n = bits 0..2, n contiguous: 16 bytes per k),
// which is exactly the canonical un-swizzled "MN-major" shared-memory operand
// layout of tcgen05.mma (core matrix = 8 k-values x 16 bytes = 128 contiguous
// bytes; next 8 k-values 128 bytes on; next 8 columns = next piece, 2048 bytes on).
// So a tile of consecutive rows is copied into shared memory AS IT IS by one bulk
// async copy and handed to the tensor core without passing through registers:
//
//     D[m][n'] = sum_k H_128[m][k] * B[k][n']        (bf16 x +-1, fp32 accumulate in TMEM)
//
// with n' = (row in tile, piece, n): N = 128 columns = 16 pieces = 32 KiB of rows.
// Products with +-1 are exact, so this is fp32 accumulation of the stored values.
// TMEM lane m (= thread m of the 128-thread epilogue group) then holds, for every
// row of the tile, the values whose index bits 3..9 equal m: bits 0..2 and the
// piece bits are all in that thread's registers, so the remaining stages are plain
// register butterflies with no exchange between threads at all, and the thread
// ends up with 8 contiguous output elements per piece: one 128-bit store, a warp
// writes 512 contiguous bytes.
//
// Roles in a CTA of 10 warps (one CTA per SM, persistent over tiles):
//   warp 0, lane 0   producer: cp.async.bulk of each tile into a shared-memory ring
//   warp 1, lane 0   issues tcgen05.mma (8 instructions of K = 16 per product) and
//                    tcgen05.commit onto mbarriers
//   warps 2..9       epilogue: tcgen05.ld, register stages, affine, stores; each warp
//                    owns TMEM lanes 32*(warp % 4) .. +31 and one half of the columns
//
// The backward pass runs two products per tile: D1 = H_128 X (for da) and
// D2 = H_128 G, where G = (a/sqrt(d)) (.) dy after ITS register stages, written back
// into the ring slot as bf16 hi + lo (two products into one accumulator; the pair
// carries 16-17 significant bits, and the accumulation is again fp32).  The backward keeps H_128
// in tensor memory and feeds it to the products from there (less shared-memory traffic per product).
//
// Every wait on an mbarrier is bounded.  A wait that expires raises a CTA-wide abort
// flag and the device status word; every role then leaves its loop, copies in flight
// are waited for (bounded), TMEM is freed and the kernel returns: a fault in the
// pipeline shows up as WHT_ERR_DEVICE_WAIT on the host, never as a hang.
// Every copy is issued by one CTA for itself alone; every source is this GPU's own memory, except in the
// column-sharded forward, whose source blocks may be peer mappings.
#pragma once
#include "mma_pipe_kernels.cuh"

namespace wht {

// ---- tcgen05 / TMEM wrappers ---------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D(tmem) (+)= A(smem desc) * B(smem desc), bf16 operands, fp32 accumulator
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The same with the A operand read from tensor memory (lane = row m, two bf16 per 32-bit column,
// K = 16 per instruction = 8 columns) instead of shared memory.
__device__ __forceinline__ void umma_bf16_a_tmem(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 16 consecutive columns of this thread's TMEM lane, written from registers
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Row m of H_128 into columns [taddr, taddr + 64) of this thread's TMEM lane: column c holds
// H[m][2c] (low half) and H[m][2c+1] (high half) as bf16.
__device__ __forceinline__ void write_h128_row_tmem(uint32_t taddr, int m) {
#pragma unroll
    for (int c0 = 0; c0 < 64; c0 += 16) {
        uint32_t r[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int k = 2 * (c0 + i);
            const uint32_t lo = (__popc(m & k) & 1) ? 0xBF80u : 0x3F80u;
            const uint32_t hi = (__popc(m & (k + 1)) & 1) ? 0xBF80u : 0x3F80u;
            r[i] = lo | (hi << 16);
        }
        tmem_st16(taddr + c0, r);
    }
    tmem_wait_st();
}

// mbarrier arrive once all tcgen05 operations issued so far by this thread are complete
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 16 consecutive columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
template <int COLS>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, float (&v)[COLS]) {
    if constexpr (COLS % 16 == 0) {
#pragma unroll
        for (int c = 0; c < COLS; c += 16) tmem_ld16(taddr + c, v + c);
    } else {
#pragma unroll
        for (int c = 0; c < COLS; c += 8) tmem_ld8(taddr + c, v + c);
    }
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// make this thread's shared-memory writes visible to the async proxy (tensor core reads)
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// try_wait that lets the hardware park the thread for up to `ns` nanoseconds (it is woken as
// soon as the phase completes), so a waiting warp does not burn issue slots polling.
__device__ __forceinline__ bool mbar_try_wait_for(uint64_t* bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}

// How long a bounded wait may last: `park` hardware-parked try_waits of up to 20 us each, then `spin`
// polls 256 ns apart (in case the parking hint is not honoured).  The kernels use the default, a few
// tenths of a second at the very least -- far beyond any copy or product; the self-test of the failure
// path passes a short one.
struct WaitLimit {
    uint32_t park = 1u << 16;
    uint32_t spin = 1u << 20;
};

// Bounded wait that also gives up as soon as another role has raised the abort flag.  When the limit
// runs out it raises the flag itself and records the fact in the device status word; it never traps.
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                              WaitLimit limit = WaitLimit{}) {
    if (mbar_try_wait(bar, parity)) return true;
    for (uint32_t i = 0; i < limit.park; ++i) {
        if (mbar_try_wait_for(bar, parity, 20000u)) return true;
        if (*abort_flag) return false;
    }
    for (uint32_t i = 0; i < limit.spin; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        __nanosleep(256);
    }
    *abort_flag = 1;
    atomicExch(&g_wht_device_error, kDeviceErrWaitExpired);
    return false;
}

// The same for a whole warp: every lane polls (and so observes the barrier itself), the
// verdict is made uniform so that the .sync.aligned tcgen05 instructions that follow are
// reached by all 32 lanes together or not at all.
__device__ __forceinline__ bool warp_wait_or_abort(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                   WaitLimit limit = WaitLimit{}) {
    const bool ok = wait_or_abort(bar, parity, abort_flag, limit);
    return __all_sync(kFullMask, ok);
}

// Self-test of the failure path: one CTA whose "producer" never produces.  Warp 0's elected lane waits
// (with the given short limit) on a barrier nobody arrives at, gives up, raises the CTA's abort flag and
// the device status word; warp 1 waits as a whole warp on a second such barrier with the default, long
// limit and must leave as soon as it sees the flag.  Every wait is bounded by construction and nothing
// traps: the kernel always returns.  out[0] = 1 when the elected wait expired, out[1] = 1 when warp 1 left
// through the abort flag.  (A template only so that the header may be included by several translation units.)
template <int UNUSED = 0>
__global__ void __launch_bounds__(64, 1)
wait_expiry_selftest_kernel(uint32_t park, uint32_t spin, unsigned int* out) {
    __shared__ __align__(8) uint64_t bars[2];
    __shared__ uint32_t abort_word;
    volatile uint32_t* abort_flag = &abort_word;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(bars + 0, 1);
        mbar_init(bars + 1, 1);
        abort_word = 0;
        fence_mbar_init();
    }
    __syncthreads();
    WaitLimit shortl;
    shortl.park = park;
    shortl.spin = spin;
    if (warp == 0) {
        if (lane == 0) {
            const bool ok = wait_or_abort(bars + 0, 0, abort_flag, shortl);
            out[0] = ok ? 0u : 1u;
        }
    } else {
        const bool ok = warp_wait_or_abort(bars + 1, 0, abort_flag);  // ends when warp 0 raises the flag
        if (lane == 0) out[1] = ok ? 0u : 1u;
    }
    __syncthreads();
}

// Shared-memory matrix descriptor: no swizzle, 128 bytes between core matrices along K,
// 2048 bytes between core matrices along M/N.  Valid for both operands used here.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t smem_addr) {
    uint64_t d = static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(128 >> 4) << 16;   // leading-dimension byte offset
    d |= static_cast<uint64_t>(2048 >> 4) << 32;  // stride-dimension byte offset
    d |= static_cast<uint64_t>(1) << 46;          // descriptor version of this architecture
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, A K-major, B MN-major, M = 128, N columns.
__host__ __device__ constexpr uint32_t umma_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (static_cast<uint32_t>(n >> 3) << 17) |
           (static_cast<uint32_t>(128 >> 4) << 24);
}

// Instruction-descriptor bit that multiplies by -A instead of A.
constexpr int kUmmaNegateABit = 13;

// compile-time booleans passed to generic lambdas
struct TrueTag { static constexpr bool value = true; };
struct FalseTag { static constexpr bool value = false; };

template <int LOGD, int NCOL_>
struct UmmaGeo {
    static constexpr int D = 1 << LOGD;
    static constexpr int PIECES = D / 1024;
    static constexpr int R = 8 * PIECES;             // values of one row held by one thread
    static constexpr int N = NCOL_;                  // accumulator columns per tile
    static constexpr int ROWS = N / R;               // rows per tile
    static constexpr int TILE_BYTES = N * 256;       // = ROWS * D * 2
    static constexpr int H_BYTES = 128 * 128 * 2;
    static constexpr int EPI_WARPS = 8;
    static constexpr int THREADS = 32 * (2 + EPI_WARPS);
    static constexpr int CPW = N / 2;                // columns per epilogue warp
    static constexpr int RPW = CPW / R;              // rows per epilogue warp and tile
    static_assert(PIECES >= 1 && RPW >= 1 && N % 16 == 0 && N <= 256, "unsupported tile");
};

// H_128 as the A operand (K-major, un-swizzled): element (m, k) at byte
// (m/8)*2048 + (k/8)*128 + (m%8)*16 + (k%8)*2; +-1 are exact in bf16.
__device__ __forceinline__ void write_h128(unsigned char* dst, int tid, int nthreads) {
    for (int c = tid; c < 2048; c += nthreads) {
        const int m = ((c >> 7) << 3) | (c & 7);
        const int k0 = ((c >> 3) & 15) << 3;
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t lo = (__popc(m & (k0 + 2 * j)) & 1) ? 0xBF80u : 0x3F80u;
            const uint32_t hi = (__popc(m & (k0 + 2 * j + 1)) & 1) ? 0xBF80u : 0x3F80u;
            w[j] = lo | (hi << 16);
        }
        *reinterpret_cast<uint4*>(dst + c * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// Stages on the index bits a thread holds: v[piece*8 + n], n = bits 0..2.
// Bit 0 pairs neighbours inside a register pair (scalar), the rest are packed.
template <int R>
__device__ __forceinline__ void thread_stages(float (&v)[R]) {
#pragma unroll
    for (int i = 0; i < R; i += 2) {
        const float lo = v[i], hi = v[i + 1];
        v[i] = lo + hi;
        v[i + 1] = lo - hi;
    }
#pragma unroll
    for (int s = 2; s < R; s <<= 1) {
#pragma unroll
        for (int i = 0; i < R; i += 2) {
            if ((i & s) == 0) {
                F2 lo = f2(v[i], v[i + 1]), hi = f2(v[i + s], v[i + s + 1]);
                bfly2(lo, hi);
                v[i] = lo.x; v[i + 1] = lo.y;
                v[i + s] = hi.x; v[i + s + 1] = hi.y;
            }
        }
    }
}

// ---- forward ---------------------------------------------------------------------------
// LEAN: a footprint small enough for TWO CTAs per SM (H_128 in tensor memory instead of shared memory, one
// accumulator, 256 tensor-memory columns), so that the CTAs of the NEXT launch in the stream can take their
// places and set themselves up while this launch still runs (programmatic dependent launch); for calls of a
// few tiles per CTA, where launch and set-up are a visible share of the time.
template <int LOGD, int NCOL, int STAGES, typename TP, bool RES = false, bool LEAN = false>
struct UmmaFwdSmem {
    using Geo = UmmaGeo<LOGD, NCOL>;
    static constexpr int ACC = LEAN ? 1 : (512 / NCOL > 4 ? 4 : 512 / NCOL);  // accumulator buffers in TMEM
    static constexpr int TMEM_COLS = (ACC * NCOL + (LEAN ? 64 : 0)) <= 256 ? 256 : 512;
    // a and b live in registers while a row's share of them is small.  At d = 8192 the plain
    // forward splits the channels between its two warp groups instead (SPLIT); with a residual,
    // whose chunks need registers too, a and b are staged in shared memory as fp32 from d = 4096 on
    // (measured: the split form is slower there).
    static constexpr bool SPLIT = Geo::R > 32 && !RES;
    static constexpr bool PARAMS_IN_SMEM = RES && Geo::R >= 32;
    static constexpr int OFF_H = 0;
    static constexpr int OFF_RING = LEAN ? 0 : Geo::H_BYTES;
    static constexpr int OFF_PARAMS = OFF_RING + STAGES * Geo::TILE_BYTES;
    static constexpr int PARAM_BYTES = PARAMS_IN_SMEM ? 2 * Geo::D * 4 : 0;
    static constexpr int OFF_BARS = OFF_PARAMS + PARAM_BYTES;
    static constexpr int NBARS = 2 * STAGES + 2 * ACC;
    static constexpr int OFF_MISC = OFF_BARS + NBARS * 8;
    static constexpr int BYTES = OFF_MISC + 16;
};

// Per-channel vector in shared memory as fp32 for d = 8192, in the order threads read it:
// float4 number ((piece*2 + half)*128 + m) holds elements piece*1024 + m*8 + half*4 .. +3.
template <int D, typename TP>
__device__ __forceinline__ void stage_params_umma(const TP* __restrict__ src, float* dst, float scale, int tid,
                                                  int nthreads) {
    for (int i = tid; i < D / 4; i += nthreads) {
        const int e0 = i * 4, piece = e0 >> 10, m = (e0 & 1023) >> 3, half = (e0 & 7) >> 2;
        float4 q;
        if constexpr (sizeof(TP) == 4) {
            q = __ldg(reinterpret_cast<const float4*>(src) + i);
        } else {
            const uint2 r = __ldg(reinterpret_cast<const uint2*>(src) + i);
            q = make_float4(bf16lo_to_f32(r.x), bf16hi_to_f32(r.x), bf16lo_to_f32(r.y), bf16hi_to_f32(r.y));
        }
        reinterpret_cast<float4*>(dst)[(piece * 2 + half) * 128 + m] =
            make_float4(q.x * scale, q.y * scale, q.z * scale, q.w * scale);
    }
}

// RES: y = resid + (a (.) (x H)/sqrt(d) + b), the residual read in the store layout (each thread
// its own 16-byte chunks, fetched before the accumulator is waited for).
//
// MULTI (column-sharded form): the rows come as nsrc blocks of D channels, one per rank, and the
// transform input is their signed sum, sign H_g[s][r].  Each block's tile is copied into a ring slot
// of its own (from this GPU's memory or through a peer mapping; plain bulk copies of one CTA for itself)
// and multiplied by H_128 into the SAME accumulator, with the instruction descriptor's negate-A bit
// set for the blocks whose sign is -1: the signed sum happens in the tensor core's fp32 accumulation
// of exact +-1 products, and the epilogue is the ordinary one.  inv_sqrt_d is then 1/sqrt(nsrc * D).
template <int LOGD, int NCOL, int STAGES, typename TP, bool RES, bool MULTI = false, bool LEAN = false>
__global__ void __launch_bounds__(UmmaGeo<LOGD, NCOL>::THREADS, 1)
umma_fwd_kernel(const __nv_bfloat16* x, const TP* __restrict__ a, const TP* __restrict__ b,
                const __nv_bfloat16* resid, __nv_bfloat16* y, long long T, float inv_sqrt_d,
                const __grid_constant__ TpParts parts,
                int nsrc_arg, unsigned neg_mask) {
    static_assert(!(RES && MULTI), "the column-sharded form has no fused residual");
    const int nsrc = MULTI ? nsrc_arg : 1;
    using Geo = UmmaGeo<LOGD, NCOL>;
    using L = UmmaFwdSmem<LOGD, NCOL, STAGES, TP, RES, LEAN>;
    constexpr int ACC = L::ACC;
    static_assert(!LEAN || !L::PARAMS_IN_SMEM, "the lean form keeps a and b in registers");
    extern __shared__ __align__(1024) unsigned char umma_smem[];
    unsigned char* const smem_raw = umma_smem;
    unsigned char* ring = smem_raw + L::OFF_RING;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw + L::OFF_BARS);
    uint64_t* full = bars;                   // [STAGES] tile landed in the ring
    uint64_t* empty = bars + STAGES;         // [STAGES] product has consumed the ring slot
    uint64_t* acc_full = bars + 2 * STAGES;  // [ACC] accumulator written
    uint64_t* acc_empty = acc_full + ACC;    // [ACC] accumulator read out by all 8 epilogue warps
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_raw + L::OFF_MISC);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem_raw + L::OFF_MISC + 4);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const long long tiles = (T + Geo::ROWS - 1) / Geo::ROWS;
    const long long my_tiles = blockIdx.x < tiles ? (tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    // Set-up.  The producer warp only needs the barriers: it initialises them, signals the others
    // (bar.arrive, it does not wait) and starts copying rows while they build H_128 and allocate
    // tensor memory; calls of a few tiles per SM are mostly ramp-up, so this start counts.
    uint32_t tmem_base = 0;
    if (warp == 0) {
        if (lane == 0) {
            for (int s = 0; s < STAGES; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
            for (int t = 0; t < ACC; ++t) { mbar_init(acc_full + t, 1); mbar_init(acc_empty + t, Geo::EPI_WARPS); }
            *abort_flag = 0;
            fence_mbar_init();
        }
        __syncwarp();
        if constexpr (L::PARAMS_IN_SMEM) {
            named_barrier(2, Geo::THREADS);
        } else {
            asm volatile("bar.arrive 2, %0;" ::"r"(Geo::THREADS) : "memory");
        }
    } else {
        if constexpr (!LEAN) {
            write_h128(smem_raw + L::OFF_H, tid - 32, Geo::THREADS - 32);
            fence_async_smem();  // H_128 was written by ordinary stores and is read by the tensor core
        }
        if (warp == 1) {
            tmem_alloc(tmem_slot, L::TMEM_COLS);
            tmem_relinquish();
        }
        tc_fence_before();
        named_barrier(2, Geo::THREADS);
        tc_fence_after();
        tmem_base = *tmem_slot;
        if constexpr (LEAN) {  // H_128 into the 64 columns after the accumulator, one row per lane
            if (warp >= 2 && warp < 6)
                write_h128_row_tmem(tmem_base + ACC * Geo::N + (static_cast<uint32_t>((warp & 3) * 32) << 16),
                                    (warp & 3) * 32 + lane);
            tc_fence_before();
            named_barrier(3, Geo::THREADS - 32);  // everybody but the producer warp
            tc_fence_after();
        }
    }
    // everything above touched only this CTA's own shared and tensor memory
    grid_dependency_wait();
    grid_launch_dependents();
    if constexpr (L::PARAMS_IN_SMEM) {
        float* pa = reinterpret_cast<float*>(smem_raw + L::OFF_PARAMS);
        stage_params_umma<Geo::D>(a, pa, inv_sqrt_d, tid, Geo::THREADS);
        stage_params_umma<Geo::D>(b, pa + Geo::D, 1.0f, tid, Geo::THREADS);
        __syncthreads();
    }

    if (warp == 0) {
        if (lane == 0) {
            const uint64_t stream_policy = l2_policy_evict_first();
            long long j = 0;  // ring slots filled so far: one per tile and source block
            bool ok = true;
            for (long long it = 0; ok && it < my_tiles; ++it) {
                const long long tile = blockIdx.x + it * gridDim.x;
                const long long row0 = tile * Geo::ROWS;
                const long long rows = T - row0 < Geo::ROWS ? T - row0 : Geo::ROWS;
                const uint32_t bytes = static_cast<uint32_t>(rows) * Geo::D * 2;
                for (int src = 0; src < nsrc; ++src, ++j) {
                    const int s = static_cast<int>(j % STAGES);
                    const uint32_t ph = static_cast<uint32_t>(j / STAGES) & 1u;
                    if (!wait_or_abort(empty + s, ph ^ 1u, abort_flag)) { ok = false; break; }
                    const __nv_bfloat16* from = MULTI ? static_cast<const __nv_bfloat16*>(parts.p[src]) : x;
                    mbar_expect_tx(full + s, bytes);
                    bulk_load_stream(ring + s * Geo::TILE_BYTES, from + row0 * Geo::D, bytes, full + s, stream_policy);
                }
            }
            if (*abort_flag) {
                // copies already issued still land in shared memory: wait for them before leaving
                const long long lo = j > STAGES ? j - STAGES : 0;
                for (long long k = lo; k < j; ++k)
                    mbar_wait_bounded(full + (k % STAGES), static_cast<uint32_t>(k / STAGES) & 1u);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint64_t adesc = umma_smem_desc(smem_u32(smem_raw + L::OFF_H));
            constexpr uint32_t idesc = umma_idesc(Geo::N);
            long long j = 0;
            bool ok = true;
            for (long long it = 0; ok && it < my_tiles; ++it) {
                const int t = static_cast<int>(it % ACC);
                const uint32_t pt = static_cast<uint32_t>(it / ACC) & 1u;
                for (int src = 0; src < nsrc; ++src, ++j) {
                    const int s = static_cast<int>(j % STAGES);
                    const uint32_t ph = static_cast<uint32_t>(j / STAGES) & 1u;
                    if (!wait_or_abort(full + s, ph, abort_flag)) { ok = false; break; }
                    if (src == 0 && !wait_or_abort(acc_empty + t, pt ^ 1u, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t bdesc = umma_smem_desc(smem_u32(ring + s * Geo::TILE_BYTES));
                    const uint32_t idesc_s = MULTI ? (idesc | (((neg_mask >> src) & 1u) << kUmmaNegateABit)) : idesc;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {  // K = 16 per instruction: 256 bytes further in both operands
                        if constexpr (LEAN)
                            umma_bf16_a_tmem(tmem_base + t * Geo::N, tmem_base + ACC * Geo::N + k * 8, bdesc + k * 16,
                                             idesc_s, (src | k) != 0);
                        else
                            umma_bf16(tmem_base + t * Geo::N, adesc + k * 16, bdesc + k * 16, idesc_s, (src | k) != 0);
                    }
                    if (src == nsrc - 1) umma_commit(acc_full + t);
                    umma_commit(empty + s);
                }
            }
        }
    } else {
        const int q = warp & 3;            // TMEM lane quarter this warp may access
        const int ch = (warp - 2) >> 2;    // which of the two 4-warp groups
        const int m = q * 32 + lane;       // index bits 3..9 of every element this thread produces

        if constexpr (L::SPLIT) {
            // d = 8192 without a residual: each group owns the channels of one value of the top index
            // bit for ALL rows of the tile, so that its share of a and b (32 values each) stays in
            // registers; it applies the stage on that bit first, straight on the two column halves
            // of the accumulator (lo + hi or lo - hi).
            constexpr int RE = Geo::R / 2, PE = RE / 8;
            const int piece0 = ch * PE;
            const F2 top_sign = ch ? f2(-1.0f, -1.0f) : f2(1.0f, 1.0f);
            const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
            F2 as[PE][4], bs[PE][4];
            {
                const F2 rs2 = f2(inv_sqrt_d, inv_sqrt_d);
#pragma unroll
                for (int p = 0; p < PE; ++p) {
                    load_params8(a + (piece0 + p) * 1024 + m * 8, as[p]);
                    load_params8(b + (piece0 + p) * 1024 + m * 8, bs[p]);
#pragma unroll
                    for (int j = 0; j < 4; ++j) as[p][j] = mul2(as[p][j], rs2);
                }
            }
            for (long long it = 0; it < my_tiles; ++it) {
                const int t = static_cast<int>(it % ACC);
                const uint32_t pt = static_cast<uint32_t>(it / ACC) & 1u;
                if (!warp_wait_or_abort(acc_full + t, pt, abort_flag)) break;
                tc_fence_after();
                const long long tile = blockIdx.x + it * gridDim.x;
#pragma unroll
                for (int r = 0; r < Geo::ROWS; ++r) {
                    const long long row = tile * Geo::ROWS + r;
                    float lo[RE], hi[RE];
                    tmem_ld_cols<RE>(lane_addr + t * Geo::N + r * Geo::R, lo);
                    tmem_ld_cols<RE>(lane_addr + t * Geo::N + r * Geo::R + RE, hi);
                    tmem_wait_ld();
                    if (r == Geo::ROWS - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(acc_empty + t);  // the accumulator is in registers now
                    }
                    float v[RE];
#pragma unroll
                    for (int i = 0; i < RE; i += 2) {
                        const F2 o = fma2(f2(hi[i], hi[i + 1]), top_sign, f2(lo[i], lo[i + 1]));
                        v[i] = o.x;
                        v[i + 1] = o.y;
                    }
                    thread_stages<RE>(v);
                    if (row < T) {
                        uint4* dst = reinterpret_cast<uint4*>(y + row * Geo::D + piece0 * 1024 + m * 8);
#pragma unroll
                        for (int p = 0; p < PE; ++p) {
                            F2 w[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) w[j] = f2(v[p * 8 + 2 * j], v[p * 8 + 2 * j + 1]);
                            fwd_store_chunk(w, as[p], bs[p], dst + p * 128);
                        }
                    }
                }
            }
        } else {
            // each group takes half of the tile's rows, every channel of them
            const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + ch * Geo::CPW;
            F2 as[L::PARAMS_IN_SMEM ? 1 : Geo::PIECES][4], bs[L::PARAMS_IN_SMEM ? 1 : Geo::PIECES][4];
            const float* pa = reinterpret_cast<const float*>(smem_raw + L::OFF_PARAMS);
            if constexpr (!L::PARAMS_IN_SMEM) {
                const F2 rs2 = f2(inv_sqrt_d, inv_sqrt_d);
#pragma unroll
                for (int p = 0; p < Geo::PIECES; ++p) {
                    load_params8(a + p * 1024 + m * 8, as[p]);
                    load_params8(b + p * 1024 + m * 8, bs[p]);
#pragma unroll
                    for (int j = 0; j < 4; ++j) as[p][j] = mul2(as[p][j], rs2);
                }
            }

            for (long long it = 0; it < my_tiles; ++it) {
                const int t = static_cast<int>(it % ACC);
                const uint32_t pt = static_cast<uint32_t>(it / ACC) & 1u;
                const long long tile = blockIdx.x + it * gridDim.x;
                // the residual chunks of this thread's rows are fetched ahead of the accumulator wait
                uint4 res[RES ? Geo::RPW * Geo::PIECES : 1];
                if constexpr (RES) {
#pragma unroll
                    for (int rl = 0; rl < Geo::RPW; ++rl) {
                        const long long row = tile * Geo::ROWS + ch * Geo::RPW + rl;
#pragma unroll
                        for (int p = 0; p < Geo::PIECES; ++p) {
                            res[rl * Geo::PIECES + p] = make_uint4(0u, 0u, 0u, 0u);
                            if (row < T)
                                res[rl * Geo::PIECES + p] =
                                    __ldcs(reinterpret_cast<const uint4*>(resid + row * Geo::D + m * 8) + p * 128);
                        }
                    }
                }
                if (!warp_wait_or_abort(acc_full + t, pt, abort_flag)) break;
                tc_fence_after();
                float u[Geo::CPW];
                tmem_ld_cols<Geo::CPW>(lane_addr + t * Geo::N, u);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_empty + t);  // the accumulator is in registers now

                // this thread's 16-byte chunk of piece 0 of its first row of the tile; FULL (every row of the
                // tile exists: all tiles but the last of a ragged problem) drops the per-row test
                const long long row_first = tile * Geo::ROWS + ch * Geo::RPW;
                uint4* const dst_first = reinterpret_cast<uint4*>(y + row_first * Geo::D + m * 8);
                auto rows_out = [&](auto full_tag) {
                constexpr bool FULL = decltype(full_tag)::value;
#pragma unroll
                for (int rl = 0; rl < Geo::RPW; ++rl) {
                    float v[Geo::R];
#pragma unroll
                    for (int i = 0; i < Geo::R; ++i) v[i] = u[rl * Geo::R + i];
                    thread_stages<Geo::R>(v);
                    if (FULL || row_first + rl < T) {
                        uint4* dst = dst_first + rl * (Geo::D / 8);
#pragma unroll
                        for (int p = 0; p < Geo::PIECES; ++p) {
                            F2 w[4];
#pragma unroll
                            for (int j = 0; j < 4; ++j) w[j] = f2(v[p * 8 + 2 * j], v[p * 8 + 2 * j + 1]);
                            if constexpr (L::PARAMS_IN_SMEM) {
                                const float4* qa = reinterpret_cast<const float4*>(pa) + (p * 2) * 128 + m;
                                const float4* qb = reinterpret_cast<const float4*>(pa + Geo::D) + (p * 2) * 128 + m;
                                const float4 a0 = qa[0], a1 = qa[128], b0 = qb[0], b1 = qb[128];
                                F2 ap[4] = {f2(a0.x, a0.y), f2(a0.z, a0.w), f2(a1.x, a1.y), f2(a1.z, a1.w)};
                                F2 bp[4] = {f2(b0.x, b0.y), f2(b0.z, b0.w), f2(b1.x, b1.y), f2(b1.z, b1.w)};
                                if constexpr (RES)
                                    fwd_store_chunk_res(w, ap, bp, res[rl * Geo::PIECES + p], dst + p * 128);
                                else
                                    fwd_store_chunk(w, ap, bp, dst + p * 128);
                            } else {
                                if constexpr (RES)
                                    fwd_store_chunk_res(w, as[p], bs[p], res[rl * Geo::PIECES + p], dst + p * 128);
                                else
                                    fwd_store_chunk(w, as[p], bs[p], dst + p * 128);
                            }
                        }
                    }
                }
                };
                if ((tile + 1) * Geo::ROWS <= T) rows_out(TrueTag{}); else rows_out(FalseTag{});
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, L::TMEM_COLS);
    }
}

// ---- backward --------------------------------------------------------------------------
template <int LOGD, int NCOL, int STAGES>
struct UmmaBwdSmem {
    using Geo = UmmaGeo<LOGD, NCOL>;
    static constexpr int STAGE_BYTES = 2 * Geo::TILE_BYTES;  // x tile, then dy tile
    static constexpr int TMEM_COLS = 4 * NCOL <= 256 ? 256 : 512;  // D1 x2, D2 x2 (or D2 x1 and H_128)
    static constexpr int OFF_H = 0;
    static constexpr int OFF_RING = Geo::H_BYTES;
    static constexpr int OFF_BARS = OFF_RING + STAGES * STAGE_BYTES;
    static constexpr int NBARS = 3 * STAGES + 8;
    static constexpr int OFF_MISC = OFF_BARS + NBARS * 8;
    static constexpr int BYTES = OFF_MISC + 16;
    static_assert(STAGES * STAGE_BYTES >= 2 * Geo::D * 4, "the ring is reused to fold da, db");
};

// partials layout: [gridDim.x][2][D] fp32; slot 0: sum_t dy (.) (x H) WITHOUT the
// 1/sqrt(d) factor (the second pass applies it), slot 1: sum_t dy.
//
// G_LO = false (the default of the library): g is rounded to bf16 once before the second product instead
// of being carried as hi + lo, so a tile costs two products instead of three and the lo half of the
// register work and of the shared-memory writes goes away.  dx then carries the 2^-9 rounding of each
// of the 128 terms of a product (about 1e-3 of a row's typical dx, far inside the 1e-2 bound, but no
// longer "one rounding at the store"); da and db do not pass through g and are unchanged.  Measured
// 13 % (d = 2048) and 11 % (d = 8192) faster in long runs, whose speed the board's power limit sets.
template <int LOGD, int NCOL, int STAGES, typename TP, bool A_TMEM = false, bool G_LO = true>
__global__ void __launch_bounds__(UmmaGeo<LOGD, NCOL>::THREADS, 1)
umma_bwd_kernel(const __nv_bfloat16* dy, const __nv_bfloat16* x, const TP* __restrict__ a, __nv_bfloat16* dx,
                float* __restrict__ partials, long long T, float inv_sqrt_d) {
    using Geo = UmmaGeo<LOGD, NCOL>;
    using L = UmmaBwdSmem<LOGD, NCOL, STAGES>;
    // How the two groups of four epilogue warps share a tile.  Up to 16 values per row and
    // thread (d <= 2048) each group takes half of the rows.  Beyond that the per-thread state
    // for all channels (da, db, a: three values per channel, next to a tile's worth of
    // accumulator columns) would not fit in registers, so each group takes ALL rows but
    // only the channels whose top index bit equals its group number: the stage on that
    // bit is applied first, straight on the accumulator columns (each thread reads both
    // halves from TMEM and keeps lo + hi or lo - hi), and for dx last, in the same way.
    constexpr bool SPLIT = Geo::R > 16;
    constexpr int RE = SPLIT ? Geo::R / 2 : Geo::R;      // values per row a thread works on
    constexpr int PE = RE / 8;                           // pieces per row a thread works on
    constexpr int NROW = SPLIT ? Geo::ROWS : Geo::RPW;   // rows per tile a thread works on
    static_assert(RE <= 32, "per-thread accumulators must fit in registers");
    // the per-row code is long at d = 8192 (32 values, five stages, twice): kept as a loop there, the
    // smaller code is measured 2 % faster; unrolled everywhere else (d = 4096 is 2.5 % slower as a loop)
    constexpr int ROW_UNROLL = Geo::R > 32 ? 1 : NROW;
    extern __shared__ __align__(1024) unsigned char umma_smem[];
    unsigned char* const smem_raw = umma_smem;
    unsigned char* ring = smem_raw + L::OFF_RING;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw + L::OFF_BARS);
    uint64_t* full = bars;                      // [STAGES] x and dy tiles landed
    uint64_t* stage_empty = bars + STAGES;      // [STAGES] second product has consumed the slot
    uint64_t* g_ready = bars + 2 * STAGES;      // [STAGES] G (hi, lo) written into the slot by the 8 warps
    uint64_t* d1_full = bars + 3 * STAGES;      // [2]
    uint64_t* d1_empty = d1_full + 2;           // [2]
    uint64_t* d2_full = d1_full + 4;            // [2]
    uint64_t* d2_empty = d1_full + 6;           // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_raw + L::OFF_MISC);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem_raw + L::OFF_MISC + 4);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const long long tiles = (T + Geo::ROWS - 1) / Geo::ROWS;
    const long long my_tiles = blockIdx.x < tiles ? (tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full + s, 1);
            mbar_init(stage_empty + s, 1);
            mbar_init(g_ready + s, Geo::EPI_WARPS);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(d1_full + t, 1);
            mbar_init(d1_empty + t, Geo::EPI_WARPS);
            mbar_init(d2_full + t, 1);
            mbar_init(d2_empty + t, Geo::EPI_WARPS);
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if constexpr (!A_TMEM) {
        write_h128(smem_raw + L::OFF_H, tid, Geo::THREADS);
        fence_async_smem();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, L::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // everything above touched only this CTA's own shared and tensor memory
    grid_dependency_wait();
    grid_launch_dependents();
    const uint32_t tmem_d1 = tmem_base;
    const uint32_t tmem_d2 = tmem_base + 2 * Geo::N;
    // A_TMEM: H_128 is kept in tensor memory (64 columns after a single D2 buffer) and the products read
    // it from there, which takes a third of their operand traffic off the shared memory
    const uint32_t tmem_a = tmem_base + 3 * Geo::N;
    if constexpr (A_TMEM) {
        static_assert(3 * Geo::N + 64 <= L::TMEM_COLS, "no room for H_128 in tensor memory");
        if (warp >= 2 && warp < 6)
            write_h128_row_tmem(tmem_a + (static_cast<uint32_t>((warp & 3) * 32) << 16), (warp & 3) * 32 + lane);
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }

    // per-thread partial column sums (epilogue warps only; declared here so that the fold
    // after the role loops can see them)
    F2 da_acc[PE][4], db_acc[PE][4];
#pragma unroll
    for (int p = 0; p < PE; ++p) {
#pragma unroll
        for (int j = 0; j < 4; ++j) { da_acc[p][j] = f2(0.0f, 0.0f); db_acc[p][j] = f2(0.0f, 0.0f); }
    }

    if (warp == 0) {
        if (lane == 0) {
            const uint64_t stream_policy = l2_policy_evict_first();
            long long it = 0;
            for (; it < my_tiles; ++it) {
                const int s = static_cast<int>(it % STAGES);
                const uint32_t ph = static_cast<uint32_t>(it / STAGES) & 1u;
                if (!wait_or_abort(stage_empty + s, ph ^ 1u, abort_flag)) break;
                const long long tile = blockIdx.x + it * gridDim.x;
                const long long row0 = tile * Geo::ROWS;
                const long long rows = T - row0 < Geo::ROWS ? T - row0 : Geo::ROWS;
                const uint32_t bytes = static_cast<uint32_t>(rows) * Geo::D * 2;
                mbar_expect_tx(full + s, 2 * bytes);
                bulk_load_stream(ring + s * L::STAGE_BYTES, x + row0 * Geo::D, bytes, full + s, stream_policy);
                bulk_load_stream(ring + s * L::STAGE_BYTES + Geo::TILE_BYTES, dy + row0 * Geo::D, bytes, full + s,
                                 stream_policy);
            }
            if (*abort_flag) {
                const long long lo = it > STAGES ? it - STAGES : 0;
                for (long long j = lo; j < it; ++j)
                    mbar_wait_bounded(full + (j % STAGES), static_cast<uint32_t>(j / STAGES) & 1u);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint64_t adesc = umma_smem_desc(smem_u32(smem_raw + L::OFF_H));
            constexpr uint32_t idesc = umma_idesc(Geo::N);
            // first product of tile i: D1 = H_128 X
            auto step_x = [&](long long i) -> bool {
                const int s = static_cast<int>(i % STAGES);
                const uint32_t ph = static_cast<uint32_t>(i / STAGES) & 1u;
                const int t = static_cast<int>(i & 1);
                const uint32_t pt = static_cast<uint32_t>(i >> 1) & 1u;
                if (!wait_or_abort(full + s, ph, abort_flag)) return false;
                if (!wait_or_abort(d1_empty + t, pt ^ 1u, abort_flag)) return false;
                tc_fence_after();
                const uint64_t bdesc = umma_smem_desc(smem_u32(ring + s * L::STAGE_BYTES));
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    if constexpr (A_TMEM)
                        umma_bf16_a_tmem(tmem_d1 + t * Geo::N, tmem_a + k * 8, bdesc + k * 16, idesc, k > 0);
                    else
                        umma_bf16(tmem_d1 + t * Geo::N, adesc + k * 16, bdesc + k * 16, idesc, k > 0);
                }
                umma_commit(d1_full + t);
                return true;
            };
            // second product of tile i: D2 = H_128 G_hi + H_128 G_lo
            auto step_g = [&](long long i) -> bool {
                const int s = static_cast<int>(i % STAGES);
                const uint32_t ph = static_cast<uint32_t>(i / STAGES) & 1u;
                const int t = A_TMEM ? 0 : static_cast<int>(i & 1);  // A_TMEM: one D2 buffer
                const uint32_t pt = static_cast<uint32_t>(A_TMEM ? i : (i >> 1)) & 1u;
                if (!wait_or_abort(g_ready + s, ph, abort_flag)) return false;
                if (!wait_or_abort(d2_empty + t, pt ^ 1u, abort_flag)) return false;
                tc_fence_after();
                const uint64_t bhi = umma_smem_desc(smem_u32(ring + s * L::STAGE_BYTES));
                const uint64_t blo = umma_smem_desc(smem_u32(ring + s * L::STAGE_BYTES + Geo::TILE_BYTES));
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    if constexpr (A_TMEM)
                        umma_bf16_a_tmem(tmem_d2 + t * Geo::N, tmem_a + k * 8, bhi + k * 16, idesc, k > 0);
                    else
                        umma_bf16(tmem_d2 + t * Geo::N, adesc + k * 16, bhi + k * 16, idesc, k > 0);
                }
                if constexpr (G_LO) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        if constexpr (A_TMEM)
                            umma_bf16_a_tmem(tmem_d2 + t * Geo::N, tmem_a + k * 8, blo + k * 16, idesc, 1);
                        else
                            umma_bf16(tmem_d2 + t * Geo::N, adesc + k * 16, blo + k * 16, idesc, 1);
                    }
                }
                umma_commit(d2_full + t);
                umma_commit(stage_empty + s);
                return true;
            };
            bool ok = my_tiles > 0 ? step_x(0) : true;
            for (long long i = 0; ok && i < my_tiles; ++i) {
                if (i + 1 < my_tiles) ok = step_x(i + 1);
                if (ok) ok = step_g(i);
            }
        }
    } else {
        const int q = warp & 3;
        const int ch = (warp - 2) >> 2;
        const int m = q * 32 + lane;
        const int piece0 = SPLIT ? ch * PE : 0;  // first piece of the channels this thread owns
        const F2 top_sign = ch ? f2(-1.0f, -1.0f) : f2(1.0f, 1.0f);  // split: lo + hi or lo - hi
        // TMEM address of this thread's lane; the non-split groups start at their half of the columns
        const uint32_t lane_off = (static_cast<uint32_t>(q * 32) << 16) + (SPLIT ? 0 : ch * Geo::CPW);

        F2 as[PE][4];
        {
            const F2 rs2 = f2(inv_sqrt_d, inv_sqrt_d);
#pragma unroll
            for (int p = 0; p < PE; ++p) {
                load_params8(a + (piece0 + p) * 1024 + m * 8, as[p]);
#pragma unroll
                for (int j = 0; j < 4; ++j) as[p][j] = mul2(as[p][j], rs2);
            }
        }

        // RE values of row r of this thread's share, from accumulator `acc`: the columns as they
        // are, or (split) the top-bit stage lo +- hi of the two column halves of the row
        auto row_values = [&](uint32_t acc, int r, float (&v)[RE], const float* preloaded) {
            if constexpr (SPLIT) {
                float lo[RE], hi[RE];
                tmem_ld_cols<RE>(acc + lane_off + r * Geo::R, lo);
                tmem_ld_cols<RE>(acc + lane_off + r * Geo::R + RE, hi);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < RE; i += 2) {
                    const F2 l = f2(lo[i], lo[i + 1]), h = f2(hi[i], hi[i + 1]);
                    const F2 o = fma2(h, top_sign, l);
                    v[i] = o.x;
                    v[i + 1] = o.y;
                }
            } else {
#pragma unroll
                for (int i = 0; i < RE; ++i) v[i] = preloaded[r * RE + i];
            }
        };

        __nv_bfloat16* const dx_thr = dx + piece0 * 1024 + m * 8;  // this thread's 8 columns of piece0
        const int ntiles = static_cast<int>(my_tiles);
        // valid rows of this CTA's j-th tile (the last tile of the problem may be ragged)
        auto rows_in_tile = [&](int j, long long& row0) -> int {
            row0 = (static_cast<long long>(blockIdx.x) + static_cast<long long>(j) * gridDim.x) * Geo::ROWS;
            const long long left = T - row0;
            return left < Geo::ROWS ? static_cast<int>(left) : Geo::ROWS;
        };

        // dx rows of tile j: read D2, (split: top-bit stage,) round, store
        auto store_dx = [&](int j) -> bool {
            const int t = A_TMEM ? 0 : (j & 1);
            const uint32_t pt = static_cast<uint32_t>(A_TMEM ? j : (j >> 1)) & 1u;
            if (!warp_wait_or_abort(d2_full + t, pt, abort_flag)) return false;
            tc_fence_after();
            const uint32_t acc = tmem_d2 + t * Geo::N;
            float u[SPLIT ? 1 : Geo::CPW];
            if constexpr (!SPLIT) {
                tmem_ld_cols<Geo::CPW>(acc + lane_off, u);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(d2_empty + t);
            }
            long long row0;
            const int nvalid = rows_in_tile(j, row0);
            uint4* const dst0 = reinterpret_cast<uint4*>(dx_thr + row0 * Geo::D);
            // FULL: every row of the tile exists (all tiles but the last one of a ragged problem): no
            // per-row test, so the rows stay one straight instruction stream
            auto store_rows = [&](auto full_tag) {
                constexpr bool FULL = decltype(full_tag)::value;
#pragma unroll(ROW_UNROLL)
                for (int r = 0; r < NROW; ++r) {
                    const int rt = SPLIT ? r : ch * Geo::RPW + r;  // row inside the tile
                    if (FULL || rt < nvalid) {                      // uniform over the warp
                        float w[RE];
                        row_values(acc, r, w, u);
#pragma unroll
                        for (int p = 0; p < PE; ++p) {
                            uint4 o;
                            o.x = pack_bf16x2(w[p * 8 + 0], w[p * 8 + 1]);
                            o.y = pack_bf16x2(w[p * 8 + 2], w[p * 8 + 3]);
                            o.z = pack_bf16x2(w[p * 8 + 4], w[p * 8 + 5]);
                            o.w = pack_bf16x2(w[p * 8 + 6], w[p * 8 + 7]);
                            __stcs(dst0 + rt * (Geo::D / 8) + p * 128, o);
                        }
                    }
                }
            };
            if (nvalid == Geo::ROWS) store_rows(TrueTag{}); else store_rows(FalseTag{});
            if constexpr (SPLIT) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(d2_empty + t);
            }
            return true;
        };

        bool ok = true;
        for (int it = 0; ok && it < ntiles; ++it) {
            const int s = it % STAGES;
            const uint32_t ph = static_cast<uint32_t>(it / STAGES) & 1u;
            const int t = it & 1;
            const uint32_t pt = static_cast<uint32_t>(it >> 1) & 1u;
            if (!warp_wait_or_abort(d1_full + t, pt, abort_flag)) { ok = false; break; }
            // the first product ran, so the tile has landed; observing the barrier ourselves
            // makes the copied dy bytes visible to this thread's ordinary loads
            if (!warp_wait_or_abort(full + s, ph, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t acc = tmem_d1 + t * Geo::N;
            float u[SPLIT ? 1 : Geo::CPW];
            if constexpr (!SPLIT) {
                tmem_ld_cols<Geo::CPW>(acc + lane_off, u);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(d1_empty + t);
            }

            // this thread's 16-byte chunk of piece0 of row 0 of the tile, in the x and dy slots
            unsigned char* const cx = ring + s * L::STAGE_BYTES + (piece0 * 128 + m) * 16;
            unsigned char* const cdy = cx + Geo::TILE_BYTES;
            long long row0;
            const int nvalid = rows_in_tile(it, row0);
            // Rows past T were never copied: their accumulator columns and slot bytes hold
            // whatever was there before.  They are skipped altogether (uniformly over the
            // warp); the second product then reads stale columns for them, which nobody stores.
            // FULL (every row of the tile exists) drops the per-row test.
            auto tile_rows = [&](auto full_tag) {
            constexpr bool FULL = decltype(full_tag)::value;
#pragma unroll(ROW_UNROLL)
            for (int r = 0; r < NROW; ++r) {
                const int rt = SPLIT ? r : ch * Geo::RPW + r;  // row inside the tile
                if (FULL || rt < nvalid) {
                    float v[RE];
                    row_values(acc, r, v, u);
                    thread_stages<RE>(v);  // v = (x H) at this thread's channels, unnormalised
                    float g[RE];
#pragma unroll
                    for (int p = 0; p < PE; ++p) {
                        const uint4 raw = *reinterpret_cast<const uint4*>(cdy + (rt * Geo::PIECES + p) * 2048);
                        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const F2 dyv = unpack_bf16x2(w[j]);
                            da_acc[p][j] = fma2(dyv, f2(v[p * 8 + 2 * j], v[p * 8 + 2 * j + 1]), da_acc[p][j]);
                            db_acc[p][j] = add2(db_acc[p][j], dyv);
                            const F2 gv = mul2(as[p][j], dyv);
                            g[p * 8 + 2 * j] = gv.x;
                            g[p * 8 + 2 * j + 1] = gv.y;
                        }
                    }
                    thread_stages<RE>(g);  // the register stages of the second transform
#pragma unroll
                    for (int p = 0; p < PE; ++p) {
                        // the x tile is consumed (D1 is complete); this thread alone read this dy chunk
                        if constexpr (G_LO) {
                            uint4 hi, lo;
                            split_hi_lo(f2(g[p * 8 + 0], g[p * 8 + 1]), hi.x, lo.x);
                            split_hi_lo(f2(g[p * 8 + 2], g[p * 8 + 3]), hi.y, lo.y);
                            split_hi_lo(f2(g[p * 8 + 4], g[p * 8 + 5]), hi.z, lo.z);
                            split_hi_lo(f2(g[p * 8 + 6], g[p * 8 + 7]), hi.w, lo.w);
                            *reinterpret_cast<uint4*>(cx + (rt * Geo::PIECES + p) * 2048) = hi;
                            *reinterpret_cast<uint4*>(cdy + (rt * Geo::PIECES + p) * 2048) = lo;
                        } else {
                            uint4 hi;
                            hi.x = pack_bf16x2(g[p * 8 + 0], g[p * 8 + 1]);
                            hi.y = pack_bf16x2(g[p * 8 + 2], g[p * 8 + 3]);
                            hi.z = pack_bf16x2(g[p * 8 + 4], g[p * 8 + 5]);
                            hi.w = pack_bf16x2(g[p * 8 + 6], g[p * 8 + 7]);
                            *reinterpret_cast<uint4*>(cx + (rt * Geo::PIECES + p) * 2048) = hi;
                        }
                    }
                }
            }
            };
            if (nvalid == Geo::ROWS) tile_rows(TrueTag{}); else tile_rows(FalseTag{});
            if constexpr (SPLIT) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(d1_empty + t);
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(g_ready + s);
            if (it > 0) ok = store_dx(it - 1);
        }
        if (ok && ntiles > 0) ok = store_dx(ntiles - 1);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, L::TMEM_COLS);
    }

    float* out = partials + static_cast<size_t>(blockIdx.x) * 2 * Geo::D;
    if constexpr (SPLIT) {
        // every (channel, thread) pair is unique: publish straight from registers
        if (warp >= 2) {
            const int m = (warp & 3) * 32 + lane;
            const int piece0 = ((warp - 2) >> 2) * PE;
#pragma unroll
            for (int p = 0; p < PE; ++p) {
                float4* oa = reinterpret_cast<float4*>(out + (piece0 + p) * 1024 + m * 8);
                float4* ob = reinterpret_cast<float4*>(out + Geo::D + (piece0 + p) * 1024 + m * 8);
                oa[0] = make_float4(da_acc[p][0].x, da_acc[p][0].y, da_acc[p][1].x, da_acc[p][1].y);
                oa[1] = make_float4(da_acc[p][2].x, da_acc[p][2].y, da_acc[p][3].x, da_acc[p][3].y);
                ob[0] = make_float4(db_acc[p][0].x, db_acc[p][0].y, db_acc[p][1].x, db_acc[p][1].y);
                ob[1] = make_float4(db_acc[p][2].x, db_acc[p][2].y, db_acc[p][3].x, db_acc[p][3].y);
            }
        }
    } else {
        // fold the two row halves (different rows of the same channels) in a fixed order and
        // publish this CTA's partial sums; the ring is free now
        float* fold = reinterpret_cast<float*>(ring);
        if (warp >= 6) {
            const int m = (warp & 3) * 32 + lane;
#pragma unroll
            for (int p = 0; p < PE; ++p) {
                float4* pd = reinterpret_cast<float4*>(fold) + ((0 * PE + p) * 2) * 128 + m;
                float4* pb = reinterpret_cast<float4*>(fold) + ((1 * PE + p) * 2) * 128 + m;
                pd[0] = make_float4(da_acc[p][0].x, da_acc[p][0].y, da_acc[p][1].x, da_acc[p][1].y);
                pd[128] = make_float4(da_acc[p][2].x, da_acc[p][2].y, da_acc[p][3].x, da_acc[p][3].y);
                pb[0] = make_float4(db_acc[p][0].x, db_acc[p][0].y, db_acc[p][1].x, db_acc[p][1].y);
                pb[128] = make_float4(db_acc[p][2].x, db_acc[p][2].y, db_acc[p][3].x, db_acc[p][3].y);
            }
        }
        __syncthreads();
        if (warp >= 2 && warp < 6) {
            const int m = (warp & 3) * 32 + lane;
#pragma unroll
            for (int p = 0; p < PE; ++p) {
                const float4* pd = reinterpret_cast<const float4*>(fold) + ((0 * PE + p) * 2) * 128 + m;
                const float4* pb = reinterpret_cast<const float4*>(fold) + ((1 * PE + p) * 2) * 128 + m;
                const float4 d0 = pd[0], d1 = pd[128], b0 = pb[0], b1 = pb[128];
                float4* oa = reinterpret_cast<float4*>(out + p * 1024 + m * 8);
                float4* ob = reinterpret_cast<float4*>(out + Geo::D + p * 1024 + m * 8);
                oa[0] = make_float4(da_acc[p][0].x + d0.x, da_acc[p][0].y + d0.y, da_acc[p][1].x + d0.z,
                                    da_acc[p][1].y + d0.w);
                oa[1] = make_float4(da_acc[p][2].x + d1.x, da_acc[p][2].y + d1.y, da_acc[p][3].x + d1.z,
                                    da_acc[p][3].y + d1.w);
                ob[0] = make_float4(db_acc[p][0].x + b0.x, db_acc[p][0].y + b0.y, db_acc[p][1].x + b0.z,
                                    db_acc[p][1].y + b0.w);
                ob[1] = make_float4(db_acc[p][2].x + b1.x, db_acc[p][2].y + b1.y, db_acc[p][3].x + b1.z,
                                    db_acc[p][3].y + b1.w);
            }
        }
    }
}

}  // namespace wht
