// tcgen05 backward of the column-sharded (tensor-parallel) form, bf16 rows, w = 1024 ... 4096 channels
// per rank, g = 2, 4 or 8 ranks.  Rank r's call computes (H_d = H_g (x) H_w, d = g*w):
//
//     z_r  = ( (sum_s H_g[s][r] x_s) H_w ) / sqrt(d)        da_r = sum_t dy_r (.) z_r,   db_r = sum_t dy_r
//     dx_r = ( (sum_s H_g[r][s] (a_s (.) dy_s)) H_w ) / sqrt(d)
//
// The x side is what the column-sharded forward does: the tile of EVERY rank's x block is copied into
// a ring slot (this GPU's memory or a peer mapping; plain bulk copies that one CTA
// issues for itself alone) and multiplied by H_128 into ONE accumulator, with the instruction descriptor's negate-A
// bit where the sign is -1, so the signed sum is the tensor core's fp32 accumulation of exact +-1
// products.  The dy side cannot be summed that way (every block has its own a_s), so each slot also
// carries the block's dy tile and the epilogue threads accumulate sum_s +- (a_s/sqrt d) (.) dy_s in
// registers as the slots arrive -- in the very layout in which the plain backward holds g.  The rank's
// own block is taken last: when it lands, D1 is complete, its dy feeds da and db, g is finished, run
// through its register stages and written over the slot as the second product's operand, exactly as in
// umma_bwd_kernel.  Per output tile: g products + one (or two), g + 1 slots of traffic in, one tile out.
//
// Roles, barriers and the bounded waits are those of umma_bwd_kernel.  A ring slot is free again when
// the tensor core has consumed its x tile (or, for the own block, the second product has consumed g)
// AND the eight epilogue warps are done with its dy tile: nine arrivals.
#pragma once
#include "umma_kernels.cuh"

namespace wht {

template <int LOGW, int NCOL, int STAGES>
struct UmmaBwdTpSmem {
    using Geo = UmmaGeo<LOGW, NCOL>;
    static constexpr int STAGE_BYTES = 2 * Geo::TILE_BYTES;  // x tile, then dy tile, of one source block
    static constexpr int TMEM_COLS = 512;                    // D1 x2, D2, H_128
    static constexpr int OFF_RING = 0;
    static constexpr int OFF_BARS = OFF_RING + STAGES * STAGE_BYTES;
    static constexpr int NBARS = 2 * STAGES + 8;
    static constexpr int OFF_MISC = OFF_BARS + NBARS * 8;
    static constexpr int BYTES = OFF_MISC + 16;
    static_assert(STAGES * STAGE_BYTES >= 2 * Geo::D * 4, "the ring is reused to fold da, db");
};

// partials layout: [gridDim.x][2][W] fp32; slot 0: sum_t dy_r (.) ((sum_s +-x_s) H_w) WITHOUT the
// 1/sqrt(d) factor (the second pass applies it), slot 1: sum_t dy_r.
template <int LOGW, int NCOL, int STAGES, typename TP, bool G_LO>
__global__ void __launch_bounds__(UmmaGeo<LOGW, NCOL>::THREADS, 1)
umma_bwd_tp_kernel(const __grid_constant__ TpParts dys, const __grid_constant__ TpParts xs,
                   const __grid_constant__ TpParts as_parts, int nsrc, int rank, unsigned neg_mask,
                   __nv_bfloat16* dx, float* __restrict__ partials, long long T, float inv_sqrt_d) {
    using Geo = UmmaGeo<LOGW, NCOL>;
    using L = UmmaBwdTpSmem<LOGW, NCOL, STAGES>;
    // as in umma_bwd_kernel: up to 16 values per row and thread each group of four epilogue warps takes
    // half of the rows; beyond that every group takes all rows and the channels of one value of the
    // top index bit
    constexpr bool SPLIT = Geo::R > 16;
    constexpr int RE = SPLIT ? Geo::R / 2 : Geo::R;
    constexpr int PE = RE / 8;
    constexpr int NROW = SPLIT ? Geo::ROWS : Geo::RPW;
    static_assert(RE <= 16 && NROW * RE <= 64, "the running sum of g must fit in registers");
    extern __shared__ __align__(1024) unsigned char umma_smem[];
    unsigned char* const smem_raw = umma_smem;
    unsigned char* ring = smem_raw + L::OFF_RING;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw + L::OFF_BARS);
    uint64_t* full = bars;                      // [STAGES] x and dy tiles of one source landed
    uint64_t* stage_empty = bars + STAGES;      // [STAGES] product and epilogue warps are done with the slot
    uint64_t* g_ready = bars + 2 * STAGES;      // [2] g (hi, lo) of a tile written by the 8 warps
    uint64_t* d1_full = g_ready + 2;            // [2]
    uint64_t* d1_empty = g_ready + 4;           // [2]
    uint64_t* d2_full = g_ready + 6;            // [1]
    uint64_t* d2_empty = g_ready + 7;           // [1]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_raw + L::OFF_MISC);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem_raw + L::OFF_MISC + 4);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const long long tiles = (T + Geo::ROWS - 1) / Geo::ROWS;
    const long long my_tiles = blockIdx.x < tiles ? (tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    // order in which a tile's source blocks pass through the ring: the rank's own block last
    auto source_of = [&](int si) { return (rank + 1 + si) % nsrc; };

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full + s, 1);
            mbar_init(stage_empty + s, 1 + Geo::EPI_WARPS);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(g_ready + t, Geo::EPI_WARPS);
            mbar_init(d1_full + t, 1);
            mbar_init(d1_empty + t, Geo::EPI_WARPS);
        }
        mbar_init(d2_full, 1);
        mbar_init(d2_empty, Geo::EPI_WARPS);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, L::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_d1 = tmem_base;
    const uint32_t tmem_d2 = tmem_base + 2 * Geo::N;
    const uint32_t tmem_a = tmem_base + 3 * Geo::N;  // H_128, 64 columns
    static_assert(3 * Geo::N + 64 <= L::TMEM_COLS, "no room for H_128 in tensor memory");
    if (warp >= 2 && warp < 6)
        write_h128_row_tmem(tmem_a + (static_cast<uint32_t>((warp & 3) * 32) << 16), (warp & 3) * 32 + lane);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    F2 da_acc[PE][4], db_acc[PE][4];
#pragma unroll
    for (int p = 0; p < PE; ++p) {
#pragma unroll
        for (int j = 0; j < 4; ++j) { da_acc[p][j] = f2(0.0f, 0.0f); db_acc[p][j] = f2(0.0f, 0.0f); }
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
                for (int si = 0; si < nsrc; ++si, ++j) {
                    const int s = static_cast<int>(j % STAGES);
                    const uint32_t ph = static_cast<uint32_t>(j / STAGES) & 1u;
                    if (!wait_or_abort(stage_empty + s, ph ^ 1u, abort_flag)) { ok = false; break; }
                    const int src = source_of(si);
                    const __nv_bfloat16* xsrc = static_cast<const __nv_bfloat16*>(xs.p[src]) + row0 * Geo::D;
                    const __nv_bfloat16* dysrc = static_cast<const __nv_bfloat16*>(dys.p[src]) + row0 * Geo::D;
                    mbar_expect_tx(full + s, 2 * bytes);
                    bulk_load_stream(ring + s * L::STAGE_BYTES, xsrc, bytes, full + s, stream_policy);
                    bulk_load_stream(ring + s * L::STAGE_BYTES + Geo::TILE_BYTES, dysrc, bytes, full + s, stream_policy);
                }
            }
            if (*abort_flag) {
                const long long lo = j > STAGES ? j - STAGES : 0;
                for (long long k = lo; k < j; ++k)
                    mbar_wait_bounded(full + (k % STAGES), static_cast<uint32_t>(k / STAGES) & 1u);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc(Geo::N);
            // second product of tile i: D2 = H_128 G_hi (+ H_128 G_lo); G lies in the slot of the tile's
            // last (own) source block
            auto g_product = [&](long long i) -> bool {
                const int tg = static_cast<int>(i & 1);
                const uint32_t ptg = static_cast<uint32_t>(i >> 1) & 1u;
                if (!wait_or_abort(g_ready + tg, ptg, abort_flag)) return false;
                if (!wait_or_abort(d2_empty, (static_cast<uint32_t>(i) & 1u) ^ 1u, abort_flag)) return false;
                tc_fence_after();
                const int s = static_cast<int>((i * nsrc + nsrc - 1) % STAGES);
                const uint64_t bhi = umma_smem_desc(smem_u32(ring + s * L::STAGE_BYTES));
#pragma unroll
                for (int k = 0; k < 8; ++k) umma_bf16_a_tmem(tmem_d2, tmem_a + k * 8, bhi + k * 16, idesc, k > 0);
                if constexpr (G_LO) {
                    const uint64_t blo = umma_smem_desc(smem_u32(ring + s * L::STAGE_BYTES + Geo::TILE_BYTES));
#pragma unroll
                    for (int k = 0; k < 8; ++k) umma_bf16_a_tmem(tmem_d2, tmem_a + k * 8, blo + k * 16, idesc, 1);
                }
                umma_commit(d2_full);
                umma_commit(stage_empty + s);
                return true;
            };
            long long j = 0;
            bool ok = true;
            for (long long it = 0; ok && it < my_tiles; ++it) {
                const int t = static_cast<int>(it & 1);
                const uint32_t pt = static_cast<uint32_t>(it >> 1) & 1u;
                for (int si = 0; ok && si < nsrc; ++si, ++j) {
                    const int s = static_cast<int>(j % STAGES);
                    const uint32_t ph = static_cast<uint32_t>(j / STAGES) & 1u;
                    if (!wait_or_abort(full + s, ph, abort_flag)) { ok = false; break; }
                    if (si == 0 && !wait_or_abort(d1_empty + t, pt ^ 1u, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t bdesc = umma_smem_desc(smem_u32(ring + s * L::STAGE_BYTES));
                    const uint32_t idesc_s = idesc | (((neg_mask >> source_of(si)) & 1u) << kUmmaNegateABit);
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        umma_bf16_a_tmem(tmem_d1 + t * Geo::N, tmem_a + k * 8, bdesc + k * 16, idesc_s, (si | k) != 0);
                    if (si == nsrc - 1) umma_commit(d1_full + t); else umma_commit(stage_empty + s);
                    // the second product of the tile before goes in here: early enough that its slot is free
                    // again before this tile's sources come round to it, late enough that g is usually ready
                    if (si == 0 && it > 0) ok = g_product(it - 1);
                }
            }
            if (ok && my_tiles > 0) g_product(my_tiles - 1);
        }
    } else {
        const int q = warp & 3;
        const int ch = (warp - 2) >> 2;
        const int m = q * 32 + lane;
        const int piece0 = SPLIT ? ch * PE : 0;
        const F2 top_sign = ch ? f2(-1.0f, -1.0f) : f2(1.0f, 1.0f);
        const uint32_t lane_off = (static_cast<uint32_t>(q * 32) << 16) + (SPLIT ? 0 : ch * Geo::CPW);
        const int own_col = piece0 * 1024 + m * 8;  // this thread's first channel

        // (a_s / sqrt(d)) with the block's sign, for this thread's channels
        auto scaled_params = [&](int src, F2 (&out)[PE][4]) {
            const float sg = ((neg_mask >> src) & 1u) ? -inv_sqrt_d : inv_sqrt_d;
            const F2 rs2 = f2(sg, sg);
#pragma unroll
            for (int p = 0; p < PE; ++p) {
                load_params8(static_cast<const TP*>(as_parts.p[src]) + own_col + p * 1024, out[p]);
#pragma unroll
                for (int j = 0; j < 4; ++j) out[p][j] = mul2(out[p][j], rs2);
            }
        };
        F2 as_own[PE][4];
        scaled_params(rank, as_own);

        // RE values of row r of this thread's share from accumulator `acc`
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

        __nv_bfloat16* const dx_thr = dx + own_col;
        const int ntiles = static_cast<int>(my_tiles);
        auto rows_in_tile = [&](int j, long long& row0) -> int {
            row0 = (static_cast<long long>(blockIdx.x) + static_cast<long long>(j) * gridDim.x) * Geo::ROWS;
            const long long left = T - row0;
            return left < Geo::ROWS ? static_cast<int>(left) : Geo::ROWS;
        };

        auto store_dx = [&](int j) -> bool {
            if (!warp_wait_or_abort(d2_full, static_cast<uint32_t>(j) & 1u, abort_flag)) return false;
            tc_fence_after();
            long long row0;
            const int nvalid = rows_in_tile(j, row0);
            uint4* const dst0 = reinterpret_cast<uint4*>(dx_thr + row0 * Geo::D);
#pragma unroll
            for (int r = 0; r < NROW; ++r) {
                const int rt = SPLIT ? r : ch * Geo::RPW + r;
                if (rt < nvalid) {  // uniform over the warp
                    float w[RE];
                    row_values(tmem_d2, r, w);
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
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(d2_empty);
            return true;
        };

        long long je = 0;  // ring slots this warp has been through
        bool ok = true;
        for (int it = 0; ok && it < ntiles; ++it) {
            const int t = it & 1;
            const uint32_t pt = static_cast<uint32_t>(it >> 1) & 1u;
            long long row0;
            const int nvalid = rows_in_tile(it, row0);
            // running sum over the source blocks of +-(a_s/sqrt d) (.) dy_s, per row of this thread's share
            F2 gsum[NROW][PE][4];
#pragma unroll
            for (int r = 0; r < NROW; ++r)
#pragma unroll
                for (int p = 0; p < PE; ++p)
#pragma unroll
                    for (int j = 0; j < 4; ++j) gsum[r][p][j] = f2(0.0f, 0.0f);

            for (int si = 0; si < nsrc - 1; ++si, ++je) {
                const int s = static_cast<int>(je % STAGES);
                const uint32_t ph = static_cast<uint32_t>(je / STAGES) & 1u;
                F2 as_s[PE][4];
                scaled_params(source_of(si), as_s);  // L1-resident after the first tiles
                // observing the barrier ourselves makes the copied bytes visible to ordinary loads
                if (!warp_wait_or_abort(full + s, ph, abort_flag)) { ok = false; break; }
                const unsigned char* const cdy =
                    ring + s * L::STAGE_BYTES + Geo::TILE_BYTES + (piece0 * 128 + m) * 16;
#pragma unroll
                for (int r = 0; r < NROW; ++r) {
                    const int rt = SPLIT ? r : ch * Geo::RPW + r;
                    if (rt < nvalid) {  // rows past T were never copied
#pragma unroll
                        for (int p = 0; p < PE; ++p) {
                            const uint4 raw = *reinterpret_cast<const uint4*>(cdy + (rt * Geo::PIECES + p) * 2048);
                            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                            for (int j = 0; j < 4; ++j) gsum[r][p][j] = fma2(as_s[p][j], unpack_bf16x2(w[j]), gsum[r][p][j]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(stage_empty + s);
            }
            if (!ok) break;

            // the rank's own block: D1 is complete once its product has run
            const int s = static_cast<int>(je % STAGES);
            const uint32_t ph = static_cast<uint32_t>(je / STAGES) & 1u;
            ++je;
            if (!warp_wait_or_abort(d1_full + t, pt, abort_flag)) { ok = false; break; }
            if (!warp_wait_or_abort(full + s, ph, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t acc = tmem_d1 + t * Geo::N;
            unsigned char* const cx = ring + s * L::STAGE_BYTES + (piece0 * 128 + m) * 16;
            unsigned char* const cdy = cx + Geo::TILE_BYTES;
#pragma unroll
            for (int r = 0; r < NROW; ++r) {
                const int rt = SPLIT ? r : ch * Geo::RPW + r;
                if (rt < nvalid) {
                    float v[RE];
                    row_values(acc, r, v);
                    thread_stages<RE>(v);  // v = ((sum_s +-x_s) H_w) at this thread's channels, unnormalised
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
                            const F2 gv = fma2(as_own[p][j], dyv, gsum[r][p][j]);
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
            tc_fence_before();
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(d1_empty + t);
                mbar_arrive(g_ready + t);
                mbar_arrive(stage_empty + s);  // our part; the second product's commit is the ninth arrival
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
        // fold the two row halves (different rows of the same channels) in a fixed order; the ring is free
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
