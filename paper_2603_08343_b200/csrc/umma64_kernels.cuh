// tcgen05 backward with half-size products, bf16 rows, d = 1024 ... 4096.
//
// In long runs the backward's speed is set by the board's power limit, that is by the energy a row
// costs, and the +-1 products are the largest on-chip share of it.  A product's multiply-adds per input
// element equal its M (every element of the B operand meets M rows of A), so the way to halve them is
// M = 64: here the tensor core takes the SIX stages on index bits 3..8 (a product with H_64) and bit 9
// joins the register stages -- one more packed add/sub per element pair and transform.
//
// Operand layout.  Inside a row, 512 consecutive elements (a "half piece": bit 9 fixed) are a 64 x 8
// matrix B[k][n] = x[8k + n], k = bits 3..8, stored exactly as the un-swizzled MN-major operand wants it
// (8 k-values x 16 bytes per core matrix, 128 bytes to the next 8 k-values), and the next half piece is
// 1024 bytes on: the descriptor's stride between column groups.  A 32 KiB tile of rows is 32 such
// column groups = 256 columns; it is multiplied in two halves of 128 columns (16 KiB of rows each).
//
// Accumulator layout.  An M = 64 accumulator occupies 16 of the 32 lanes of each quarter of tensor
// memory (row i in lane 32*(i/16) + i%16), and a second one may sit in the other 16 (lane offset 16):
// the first half of the tile goes to the lower lanes, the second half to the upper ones, into the SAME
// 128 columns.  Epilogue thread (quarter q, lane l) therefore owns index bits 3..8 = 16q + l%16 of the rows
// of tile half l/16, all 128 lanes and columns are in use, and the per-thread work is that of the
// full-size kernel: the values of a row with its bits 3..8 fixed -- now 16 per 1024 elements, bits 0..2
// and 9 and the piece bits -- pass through the register stages, and 8 contiguous elements (one 128-bit
// access) come out per half piece.
//
// Everything else -- roles, ring, barriers, bounded waits, the hi (+ lo) write-back of g into the consumed
// slot, per-CTA partial sums -- is umma_bwd_kernel's.  Rows of a ragged last tile: the two halves of a
// warp hold different rows, so nothing warp-synchronous may depend on a row being valid; such rows are
// computed on whatever the slot holds and only their accumulation and their stores are masked.
#pragma once
#include "umma_kernels.cuh"

namespace wht {

template <int LOGD>
struct Umma64Geo {
    static constexpr int D = 1 << LOGD;
    static constexpr int HP = D / 512;               // half pieces per row
    static constexpr int R = 8 * HP;                 // values of one row held by one thread: 16 per 1024 elements
    static constexpr int N = 128;                    // accumulator columns (per half of the tile)
    static constexpr int ROWS_HALF = N / R;          // rows per tile half
    static constexpr int ROWS = 2 * ROWS_HALF;       // rows per tile
    static constexpr int TILE_BYTES = ROWS * D * 2;  // 32 KiB
    static constexpr int HALF_BYTES = TILE_BYTES / 2;
    static constexpr int H_BYTES = 64 * 64 * 2;
    static constexpr int EPI_WARPS = 8;
    static constexpr int THREADS = 32 * (2 + EPI_WARPS);
    static constexpr int CPW = N / 2;                // columns per epilogue warp group (rows split)
    static_assert(HP >= 2 && ROWS_HALF >= 1 && TILE_BYTES == 32768, "unsupported width");
};

template <int LOGD, int STAGES>
struct Umma64BwdSmem {
    using Geo = Umma64Geo<LOGD>;
    static constexpr int STAGE_BYTES = 2 * Geo::TILE_BYTES;  // x tile, then dy tile
    static constexpr int TMEM_COLS = 512;                    // D1 x2, D2
    static constexpr int OFF_H = 0;
    static constexpr int OFF_RING = Geo::H_BYTES;
    static constexpr int OFF_BARS = OFF_RING + STAGES * STAGE_BYTES;
    static constexpr int NBARS = 3 * STAGES + 8;
    static constexpr int OFF_MISC = OFF_BARS + NBARS * 8;
    static constexpr int BYTES = OFF_MISC + 16;
    static_assert(STAGES * STAGE_BYTES >= 4 * 2 * Geo::D * 4, "the ring is reused to fold da, db");
};

// H_64 as the A operand (K-major, un-swizzled): element (m, k) at byte
// (m/8)*1024 + (k/8)*128 + (m%8)*16 + (k%8)*2.
__device__ __forceinline__ void write_h64(unsigned char* dst, int tid, int nthreads) {
    for (int c = tid; c < 512; c += nthreads) {  // 16-byte chunk c: rows m, eight k
        const int m = ((c >> 6) << 3) | (c & 7);
        const int k0 = ((c >> 3) & 7) << 3;
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

// Shared-memory matrix descriptor for K = 64 operands: 128 bytes between core matrices along K,
// 1024 bytes between core matrices along M/N.
__device__ __forceinline__ uint64_t umma64_smem_desc(uint32_t smem_addr) {
    uint64_t d = static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>(128 >> 4) << 16;
    d |= static_cast<uint64_t>(1024 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, A K-major, B MN-major, M = 64, N columns.
__host__ __device__ constexpr uint32_t umma64_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (static_cast<uint32_t>(n >> 3) << 17) |
           (static_cast<uint32_t>(64 >> 4) << 24);
}
// the second M = 64 accumulator of a column range: the upper 16 lanes of every quarter
constexpr uint32_t kTmemUpperHalfLanes = 16u << 16;

// partials layout: [gridDim.x][2][D] fp32; slot 0: sum_t dy (.) (x H) WITHOUT the 1/sqrt(d) factor
// (the second pass applies it), slot 1: sum_t dy.
template <int LOGD, int STAGES, typename TP, bool G_LO>
__global__ void __launch_bounds__(Umma64Geo<LOGD>::THREADS, 1)
umma64_bwd_kernel(const __nv_bfloat16* dy, const __nv_bfloat16* x, const TP* __restrict__ a, __nv_bfloat16* dx,
                  float* __restrict__ partials, long long T, float inv_sqrt_d) {
    using Geo = Umma64Geo<LOGD>;
    using L = Umma64BwdSmem<LOGD, STAGES>;
    // Up to 16 values per row and thread, the two groups of four epilogue warps take different rows of
    // their tile half.  Beyond that each group takes all rows but only the channels whose top index bit
    // equals its group number, applying the stage on that bit first, straight on the two column halves
    // of a row (and for dx last, in the same way).
    constexpr bool SPLIT = Geo::R > 16;
    constexpr int RE = SPLIT ? Geo::R / 2 : Geo::R;          // values per row a thread works on
    constexpr int PE = RE / 8;                               // half pieces per row a thread works on
    constexpr int NROW = SPLIT ? Geo::ROWS_HALF : Geo::CPW / Geo::R;  // rows per tile a thread works on
    static_assert(RE <= 32 && NROW >= 1, "per-thread accumulators must fit in registers");
    extern __shared__ __align__(1024) unsigned char umma_smem[];
    unsigned char* const smem_raw = umma_smem;
    unsigned char* ring = smem_raw + L::OFF_RING;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw + L::OFF_BARS);
    uint64_t* full = bars;                      // [STAGES] x and dy tiles landed
    uint64_t* stage_empty = bars + STAGES;      // [STAGES] second product has consumed the slot
    uint64_t* g_ready = bars + 2 * STAGES;      // [STAGES] g written into the slot by the 8 warps
    uint64_t* d1_full = bars + 3 * STAGES;      // [2]
    uint64_t* d1_empty = d1_full + 2;           // [2]
    uint64_t* d2_full = d1_full + 4;            // [1]
    uint64_t* d2_empty = d1_full + 6;           // [1]
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
        }
        mbar_init(d2_full, 1);
        mbar_init(d2_empty, Geo::EPI_WARPS);
        *abort_flag = 0;
        fence_mbar_init();
    }
    write_h64(smem_raw + L::OFF_H, tid, Geo::THREADS);
    fence_async_smem();  // H_64 was written by ordinary stores and is read by the tensor core
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
            const uint64_t adesc = umma64_smem_desc(smem_u32(smem_raw + L::OFF_H));
            constexpr uint32_t idesc = umma64_idesc(Geo::N);
            // H_64 times both halves of the tile at `src` (K = 64: four instructions of K = 16 each, 256 bytes
            // further in both operands), the second half into the upper lanes
            auto products = [&](uint32_t d_tmem, const unsigned char* src, bool accumulate) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const uint64_t bdesc = umma64_smem_desc(smem_u32(src + half * Geo::HALF_BYTES));
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_bf16(d_tmem + half * kTmemUpperHalfLanes, adesc + k * 16, bdesc + k * 16, idesc,
                                  (accumulate || k > 0) ? 1u : 0u);
                }
            };
            auto step_x = [&](long long i) -> bool {  // first product of tile i: D1 = H_64 X
                const int s = static_cast<int>(i % STAGES);
                const uint32_t ph = static_cast<uint32_t>(i / STAGES) & 1u;
                const int t = static_cast<int>(i & 1);
                const uint32_t pt = static_cast<uint32_t>(i >> 1) & 1u;
                if (!wait_or_abort(full + s, ph, abort_flag)) return false;
                if (!wait_or_abort(d1_empty + t, pt ^ 1u, abort_flag)) return false;
                tc_fence_after();
                products(tmem_d1 + t * Geo::N, ring + s * L::STAGE_BYTES, false);
                umma_commit(d1_full + t);
                return true;
            };
            auto step_g = [&](long long i) -> bool {  // second product of tile i: D2 = H_64 G_hi (+ H_64 G_lo)
                const int s = static_cast<int>(i % STAGES);
                const uint32_t ph = static_cast<uint32_t>(i / STAGES) & 1u;
                if (!wait_or_abort(g_ready + s, ph, abort_flag)) return false;
                if (!wait_or_abort(d2_empty, (static_cast<uint32_t>(i) & 1u) ^ 1u, abort_flag)) return false;
                tc_fence_after();
                products(tmem_d2, ring + s * L::STAGE_BYTES, false);
                if constexpr (G_LO) products(tmem_d2, ring + s * L::STAGE_BYTES + Geo::TILE_BYTES, true);
                umma_commit(d2_full);
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
        const int hs = lane >> 4;               // which half of the tile this thread's lane holds
        const int m = q * 16 + (lane & 15);     // index bits 3..8 of every element this thread produces
        const int hp0 = SPLIT ? ch * PE : 0;    // first half piece of the channels this thread owns
        const F2 top_sign = ch ? f2(-1.0f, -1.0f) : f2(1.0f, 1.0f);
        // TMEM address of this warp's lane quarter; the non-split groups start at their rows' columns
        const uint32_t lane_off = (static_cast<uint32_t>(q * 32) << 16) + (SPLIT ? 0 : ch * Geo::CPW);
        // first row (inside the tile) of this thread's share
        const int row_first = hs * Geo::ROWS_HALF + (SPLIT ? 0 : ch * NROW);

        F2 as[PE][4];
        {
            const F2 rs2 = f2(inv_sqrt_d, inv_sqrt_d);
#pragma unroll
            for (int p = 0; p < PE; ++p) {
                load_params8(a + (hp0 + p) * 512 + m * 8, as[p]);
#pragma unroll
                for (int j = 0; j < 4; ++j) as[p][j] = mul2(as[p][j], rs2);
            }
        }

        // RE values of local row r from accumulator `acc` (warp-synchronous: every lane takes part)
        auto row_values = [&](uint32_t acc, int r, float (&v)[RE]) {
            if constexpr (SPLIT) {
                float lo[RE], hi[RE];
                tmem_ld_cols<RE>(acc + lane_off + r * Geo::R, lo);
                tmem_ld_cols<RE>(acc + lane_off + r * Geo::R + RE, hi);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < RE; i += 2) {
                    const F2 o = fma2(f2(hi[i], hi[i + 1]), top_sign, f2(lo[i], lo[i + 1]));
                    v[i] = o.x;
                    v[i + 1] = o.y;
                }
            } else {
                tmem_ld_cols<RE>(acc + lane_off + r * RE, v);
                tmem_wait_ld();
            }
        };

        __nv_bfloat16* const dx_thr = dx + hp0 * 512 + m * 8;  // this thread's 8 columns of its first half piece
        const int ntiles = static_cast<int>(my_tiles);
        auto rows_in_tile = [&](int j, long long& row0) -> int {
            row0 = (static_cast<long long>(blockIdx.x) + static_cast<long long>(j) * gridDim.x) * Geo::ROWS;
            const long long left = T - row0;
            return left < Geo::ROWS ? static_cast<int>(left) : Geo::ROWS;
        };

        // dx rows of tile j: read D2, (split: top-bit stage,) round, store
        auto store_dx = [&](int j) -> bool {
            if (!warp_wait_or_abort(d2_full, static_cast<uint32_t>(j) & 1u, abort_flag)) return false;
            tc_fence_after();
            long long row0;
            const int nvalid = rows_in_tile(j, row0);
            uint4* const dst0 = reinterpret_cast<uint4*>(dx_thr + row0 * Geo::D);
            // FULL: every row of the tile exists (all tiles but the last one of a ragged problem)
            auto store_rows = [&](auto full_tag) {
                constexpr bool FULL = decltype(full_tag)::value;
#pragma unroll
                for (int r = 0; r < NROW; ++r) {
                    const int rt = row_first + r;
                    float w[RE];
                    row_values(tmem_d2, r, w);
                    if (FULL || rt < nvalid) {  // per lane: the halves of a warp hold different rows
#pragma unroll
                        for (int p = 0; p < PE; ++p) {
                            uint4 o;
                            o.x = pack_bf16x2(w[p * 8 + 0], w[p * 8 + 1]);
                            o.y = pack_bf16x2(w[p * 8 + 2], w[p * 8 + 3]);
                            o.z = pack_bf16x2(w[p * 8 + 4], w[p * 8 + 5]);
                            o.w = pack_bf16x2(w[p * 8 + 6], w[p * 8 + 7]);
                            __stcs(dst0 + rt * (Geo::D / 8) + p * 64, o);
                        }
                    }
                }
            };
            if (nvalid == Geo::ROWS) store_rows(TrueTag{}); else store_rows(FalseTag{});
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(d2_empty);
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
            // this thread's 16-byte chunk of its first half piece of row 0 of the tile, in the x and dy slots
            unsigned char* const cx = ring + s * L::STAGE_BYTES + hp0 * 1024 + m * 16;
            unsigned char* const cdy = cx + Geo::TILE_BYTES;
            long long row0;
            const int nvalid = rows_in_tile(it, row0);
            // Rows past T were never copied: their accumulator columns and slot bytes hold whatever was
            // there before.  They are computed all the same (the loads from tensor memory are
            // warp-wide) and kept out of the column sums; the second product reads stale columns for
            // them, which nobody stores.  FULL (every row of the tile exists) drops the test.
            auto tile_rows = [&](auto full_tag) {
            constexpr bool FULL = decltype(full_tag)::value;
#pragma unroll
            for (int r = 0; r < NROW; ++r) {
                const int rt = row_first + r;
                const bool valid = FULL || rt < nvalid;
                float v[RE];
                row_values(acc, r, v);
                thread_stages<RE>(v);  // v = (x H) at this thread's channels, unnormalised
                float g[RE];
#pragma unroll
                for (int p = 0; p < PE; ++p) {
                    const uint4 raw = *reinterpret_cast<const uint4*>(cdy + (rt * Geo::HP + p) * 1024);
                    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const F2 dyv = unpack_bf16x2(w[j]);
                        if (valid) {
                            da_acc[p][j] = fma2(dyv, f2(v[p * 8 + 2 * j], v[p * 8 + 2 * j + 1]), da_acc[p][j]);
                            db_acc[p][j] = add2(db_acc[p][j], dyv);
                        }
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
                        *reinterpret_cast<uint4*>(cx + (rt * Geo::HP + p) * 1024) = hi;
                        *reinterpret_cast<uint4*>(cdy + (rt * Geo::HP + p) * 1024) = lo;
                    } else {
                        uint4 hi;
                        hi.x = pack_bf16x2(g[p * 8 + 0], g[p * 8 + 1]);
                        hi.y = pack_bf16x2(g[p * 8 + 2], g[p * 8 + 3]);
                        hi.z = pack_bf16x2(g[p * 8 + 4], g[p * 8 + 5]);
                        hi.w = pack_bf16x2(g[p * 8 + 6], g[p * 8 + 7]);
                        *reinterpret_cast<uint4*>(cx + (rt * Geo::HP + p) * 1024) = hi;
                    }
                }
            }
            };
            if (nvalid == Geo::ROWS) tile_rows(TrueTag{}); else tile_rows(FalseTag{});
            tc_fence_before();
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(d1_empty + t);
                mbar_arrive(g_ready + s);
            }
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

    // Threads that hold the same channels for different rows (the two tile halves; without the channel
    // split also the two warp groups) are folded through the ring, now free, in a fixed order.
    constexpr int NFOLD = SPLIT ? 2 : 4;
    float* fold = reinterpret_cast<float*>(ring);  // [NFOLD][2][D]
    if (warp >= 2) {
        const int ch = (warp - 2) >> 2;
        const int hs = lane >> 4;
        const int m = (warp & 3) * 16 + (lane & 15);
        const int hp0 = SPLIT ? ch * PE : 0;
        const int slot = SPLIT ? hs : ch * 2 + hs;
#pragma unroll
        for (int p = 0; p < PE; ++p) {
            float4* pd = reinterpret_cast<float4*>(fold + (slot * 2 + 0) * Geo::D + (hp0 + p) * 512 + m * 8);
            float4* pb = reinterpret_cast<float4*>(fold + (slot * 2 + 1) * Geo::D + (hp0 + p) * 512 + m * 8);
            pd[0] = make_float4(da_acc[p][0].x, da_acc[p][0].y, da_acc[p][1].x, da_acc[p][1].y);
            pd[1] = make_float4(da_acc[p][2].x, da_acc[p][2].y, da_acc[p][3].x, da_acc[p][3].y);
            pb[0] = make_float4(db_acc[p][0].x, db_acc[p][0].y, db_acc[p][1].x, db_acc[p][1].y);
            pb[1] = make_float4(db_acc[p][2].x, db_acc[p][2].y, db_acc[p][3].x, db_acc[p][3].y);
        }
    }
    __syncthreads();
    float* out = partials + static_cast<size_t>(blockIdx.x) * 2 * Geo::D;
    for (int j = tid; j < 2 * Geo::D; j += Geo::THREADS) {  // j = which * D + channel
        float sum = 0.0f;
#pragma unroll
        for (int k = 0; k < NFOLD; ++k) sum += fold[k * 2 * Geo::D + j];
        out[j] = sum;
    }
}

}  // namespace wht
