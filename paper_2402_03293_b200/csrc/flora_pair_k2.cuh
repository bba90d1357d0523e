// Decompression fused with the update for ranks above 64 on CTA pairs (tcgen05.mma.cta_group::2):  W <- W - step * S A.
//
// Same structure as decompress_tc_kernel (a slab of 128 columns of A stays resident while the row tiles of W stream
// past it), with two CTAs working on one slab: an MMA multiplies the 128 rows of the sketch tile of either CTA
// (M = 256) with the slab, of which each CTA generates and holds only the 64 columns that the instruction takes
// from its shared memory (the N x K operand is split over the pair).  Half a slab is 32 KB at r = 256, so two
// buffers fit and the slab of the next item is generated while the current item streams, which a single CTA
// cannot do above r = 192.  The pair takes the row tiles of an item in turn (the leader the even ones), so an item
// streams in half the time and each CTA generates half as much per item.  Each CTA loads, combines and stores its
// own W tiles; the leader's one thread issues the MMAs for both and learns from a relay thread of the follower
// that the follower's sketch chunks have landed.
// The sketch is read from its bf16 copy (see sketch_to_bf16_kernel).  All waits are bounded.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "flora_ptx.cuh"
#include "flora_rng.cuh"
#include "flora_tc.cuh"

namespace flora {

constexpr int K2P_FIXED_WARPS = 12;   // warp 0: W loads, 1: MMA issue (leader) / relay (follower), 2-5 and 8-11: combine, 6: S loads, 7: W stores
constexpr int K2P_GEN_WARPS = 8;      // warps 12..19: slab generators
constexpr int K2P_THREADS = 32 * (K2P_FIXED_WARPS + K2P_GEN_WARPS);
constexpr int K2P_BN = 128;           // columns of a slab (64 per CTA)

struct K2PairSmem {
    uint64_t w_full[K2_MAX_SLOTS], w_free[K2_MAX_SLOTS], out_ready[K2_MAX_SLOTS];
    uint64_t c_full[K2_MAX_CSTAGES], c_empty[K2_MAX_CSTAGES], acc_full[2], acc_empty[2], slab_full[2], slab_empty[2];
    uint32_t tmem_base;
    int abort;
};

// Cluster c (two CTAs) processes the items c, c + clusters, ...; within an item, tile iteration p covers the row tiles
// 2p (leader) and 2p + 1 (follower; it may not exist, then the follower loads and stores nothing for that iteration).
__global__ void __launch_bounds__(K2P_THREADS, 1)
decompress_pair_kernel(const TcMatrix* __restrict__ mats, const K2Item* __restrict__ items, int n_items, const __grid_constant__ SeedTable seeds,
                       int seed_base, int r, float scale, float step, int slots, int cstages)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    const int kchunks = (r + 63) >> 6;                          // 64 values of the rank per 128-byte row of bf16
    const uint32_t slab_block = 64u * 128u;                     // one K chunk of this CTA's half of a slab: 64 columns of W
    const uint32_t slab_bytes = (uint32_t)kchunks * slab_block;
    const uint32_t slab0 = smem_base;
    const uint32_t c_ring = slab0 + 2u * slab_bytes;
    const uint32_t w_ring = c_ring + (uint32_t)cstages * (uint32_t)S_CHUNK_BYTES;
    const uint32_t slot_bytes = 2u * (uint32_t)W_BOX_BYTES;     // a W tile: two boxes of 64 columns
    K2PairSmem* ctl = reinterpret_cast<K2PairSmem*>(smem_raw + (w_ring - ptx::smem_addr(smem_raw)) + (size_t)slots * slot_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t half = ptx::cluster_ctarank();
    const int cluster = (int)(blockIdx.x >> 1), clusters = (int)(gridDim.x >> 1);
    const uint32_t tmem_cols = 2u * K2P_BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < slots; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->w_full[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->w_free[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->out_ready[s]), 8);
        }
        for (int s = 0; s < cstages; ++s) {
            // the leader's barrier of a stage also takes the follower's word that its own chunk has landed: one wait per chunk
            ptx::mbar_init(ptx::smem_addr(&ctl->c_full[s]), half == 0 ? 2 : 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->c_empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_full[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_empty[s]), 16);                 // the eight combine warps of both CTAs (leader's barrier)
            ptx::mbar_init(ptx::smem_addr(&ctl->slab_full[s]), 2 * K2P_GEN_WARPS);  // the generator warps of both CTAs (leader's barrier)
            ptx::mbar_init(ptx::smem_addr(&ctl->slab_empty[s]), 1);
        }
        ctl->abort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_addr(&ctl->tmem_base), tmem_cols);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                    // both CTAs' barriers exist before either arrives on the other's
    ptx::tc_fence_after_sync();
    const uint32_t tmem = ctl->tmem_base;
    volatile int* abort = &ctl->abort;
    // tile iterations of an item, and whether this CTA has a tile in iteration p
    auto iterations = [](const K2Item& it) { return (it.tiles + 1) >> 1; };
    auto has_tile = [&](const K2Item& it, int p) { return 2 * p + (int)half < it.tiles; };

    if (warp == 0) {
        // ------------------------------------------------------------------ W tile loads
        if (lane == 0) {
            RingPos pw;
            int issued = 0;
            bool ok = true;
            for (int it = cluster; it < n_items && ok; it += clusters) {
                const K2Item item = items[it];
                const TcMatrix* mat = mats + item.mat;
                const int live_boxes = min(2, (mat->m - item.col0 + 63) >> 6);
                for (int p = 0; p < iterations(item); ++p, pw.advance(slots), ++issued) {
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->w_free[pw.s]), (pw.wraps & 1u) ^ 1u, abort);
                    if (!ok) break;
                    const uint32_t bar = ptx::smem_addr(&ctl->w_full[pw.s]);
                    if (has_tile(item, p)) {
                        ptx::mbar_arrive_expect_tx(bar, (uint32_t)live_boxes * W_BOX_BYTES);
                        for (int bx = 0; bx < live_boxes; ++bx)
                            ptx::tma_load_2d(w_ring + pw.s * slot_bytes + bx * W_BOX_BYTES, &mat->map_w, item.col0 + bx * 64, item.row0 + (2 * p + (int)half) * 128, bar);
                    } else {
                        ptx::mbar_arrive(bar);
                    }
                }
            }
            if (*abort)   // loads that nobody consumed: wait (bounded) until they have landed
                for (int g = max(0, issued - slots); g < issued; ++g) ptx::mbar_wait(ptx::smem_addr(&ctl->w_full[g % slots]), (uint32_t)(g / slots) & 1u, abort);
        }
    } else if (warp == 6) {
        // ------------------------------------------------------------------ S chunk loads (bf16 copy, 64 values of the rank each)
        if (lane == 0) {
            RingPos pc;
            bool ok = true;
            for (int it = cluster; it < n_items && ok; it += clusters) {
                const K2Item item = items[it];
                const TcMatrix* mat = mats + item.mat;
                for (int p = 0; p < iterations(item) && ok; ++p) {
                    for (int kc = 0; kc < kchunks; ++kc, pc.advance(cstages)) {
                        ok = ptx::mbar_wait(ptx::smem_addr(&ctl->c_empty[pc.s]), (pc.wraps & 1u) ^ 1u, abort);
                        if (!ok) break;
                        const uint32_t bar = ptx::smem_addr(&ctl->c_full[pc.s]);
                        if (has_tile(item, p)) {
                            ptx::mbar_arrive_expect_tx(bar, S_CHUNK_BYTES);
                            ptx::tma_load_2d(c_ring + pc.s * S_CHUNK_BYTES, &mat->map_sb, kc * 64, item.row0 + (2 * p + (int)half) * 128, bar);
                        } else {
                            ptx::mbar_arrive(bar);
                        }
                    }
                }
            }
            if (*abort)
                for (int s = 0; s < cstages; ++s) {
                    const uint32_t fills = pc.wraps + (s < pc.s ? 1u : 0u);
                    if (fills) ptx::mbar_wait(ptx::smem_addr(&ctl->c_full[s]), (fills - 1u) & 1u, abort);
                }
        }
    } else if (warp == 1) {
        if (lane == 0 && half == 0) {
            // -------------------------------------------------------------- MMA issuer (the pair's leader)
            const uint32_t idesc = ptx::umma_idesc_bf16_mn(256u, (uint32_t)K2P_BN);
            const uint64_t desc_ring = ptx::umma_desc_k_sw128(c_ring);
            RingPos pc;
            int gt = 0, k = 0;
            bool ok = true;
            for (int it = cluster; it < n_items && ok; it += clusters, ++k) {
                const K2Item item = items[it];
                const int sb = k & 1;
                const uint64_t desc_slab = ptx::umma_desc_k_sw128(slab0 + sb * slab_bytes);
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->slab_full[sb]), (uint32_t)(k >> 1) & 1u, abort);     // both halves of the slab are written
                for (int p = 0; p < iterations(item) && ok; ++p, ++gt) {
                    const uint32_t acc_addr = tmem + (uint32_t)(gt & 1) * K2P_BN;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_empty[gt & 1]), (((uint32_t)gt >> 1) & 1u) ^ 1u, abort);
                    for (int kc = 0; kc < kchunks && ok; ++kc, pc.advance(cstages)) {
                        const int s = pc.s;
                        ok = ptx::mbar_wait(ptx::smem_addr(&ctl->c_full[s]), pc.wraps & 1u, abort);
                        if (!ok) break;
                        ptx::tc_fence_after_sync();
#pragma unroll
                        for (int k16 = 0; k16 < 4; ++k16) {
                            // descriptors differ from the ring / slab base only in the start-address field (16-byte units); the
                            // same offsets address the follower's chunk and its half of the slab
                            const uint64_t da = desc_ring + (uint64_t)((s * S_CHUNK_BYTES + k16 * 32) >> 4);
                            const uint64_t db = desc_slab + (uint64_t)((kc * slab_block + k16 * 32) >> 4);
                            ptx::umma_bf16_pair(acc_addr, da, db, idesc, (kc | k16) != 0);
                        }
                        ptx::umma_commit_pair(ptx::smem_addr(&ctl->c_empty[s]), (uint16_t)3u);
                    }
                    if (ok) ptx::umma_commit_pair(ptx::smem_addr(&ctl->acc_full[gt & 1]), (uint16_t)3u);
                }
                if (ok) ptx::umma_commit_pair(ptx::smem_addr(&ctl->slab_empty[sb]), (uint16_t)3u);   // every MMA that reads this slab has completed
            }
        } else if (lane == 0) {
            // -------------------------------------------------------------- relay (the follower): its sketch chunk has landed
            RingPos pc;
            bool ok = true;
            for (int it = cluster; it < n_items && ok; it += clusters) {
                const K2Item item = items[it];
                for (int c = 0; c < iterations(item) * kchunks; ++c, pc.advance(cstages)) {
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->c_full[pc.s]), pc.wraps & 1u, abort);
                    if (!ok) break;
                    ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_addr(&ctl->c_full[pc.s]), 0u));
                }
            }
        }
    } else if (warp == 7) {
        // ------------------------------------------------------------------ W tile stores
        if (lane == 0) {
            RingPos pw;
            bool ok = true;
            for (int it = cluster; it < n_items && ok; it += clusters) {
                const K2Item item = items[it];
                const TcMatrix* mat = mats + item.mat;
                const int live_boxes = min(2, (mat->m - item.col0 + 63) >> 6);
                for (int p = 0; p < iterations(item); ++p, pw.advance(slots)) {
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->out_ready[pw.s]), pw.wraps & 1u, abort);
                    if (!ok) break;
                    if (has_tile(item, p)) {
                        for (int bx = 0; bx < live_boxes; ++bx)
                            ptx::tma_store_2d(&mat->map_w, item.col0 + bx * 64, item.row0 + (2 * p + (int)half) * 128, w_ring + pw.s * slot_bytes + bx * W_BOX_BYTES);
                        ptx::tma_store_commit();
                        ptx::tma_store_wait_read<0>();          // the slot has been read out: it can be refilled
                    }
                    ptx::mbar_arrive(ptx::smem_addr(&ctl->w_free[pw.s]));
                }
            }
            ptx::tma_store_wait_all<0>();
        }
    } else if ((warp >= 2 && warp <= 5) || (warp >= 8 && warp <= 11)) {
        // ------------------------------------------------------------------ combine the accumulator with the W tile
        // Eight warps: warp w owns tensor-memory lanes 32*(w%4) .. +31 (rows of this CTA's tile); warps 2-5 take the
        // left 64 columns of the tile, warps 8-11 the right 64.  All accumulator loads of a warp are issued before the
        // first is consumed.
        const int quarter = warp & 3;
        const int side = warp >= 8 ? 1 : 0;
        const int row = quarter * 32 + lane;
        RingPos pw;
        int gt = 0;
        bool ok = true;
        for (int it = cluster; it < n_items && ok; it += clusters) {
            const K2Item item = items[it];
            const int live_chunks = min(2, (mats[item.mat].m - item.col0 + 63) >> 6) << 2;     // 16-column chunks that hold columns of W
            const int c_begin = side * 4;
            const int mine = max(0, min(4, live_chunks - c_begin));
            for (int p = 0; p < iterations(item); ++p, ++gt, pw.advance(slots)) {
                const int s = pw.s;
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_full[gt & 1]), ((uint32_t)gt >> 1) & 1u, abort) &&
                     ptx::mbar_wait(ptx::smem_addr(&ctl->w_full[s]), pw.wraps & 1u, abort);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                if (has_tile(item, p)) {
                    const uint32_t wrow = w_ring + s * slot_bytes + row * 128;
                    uint32_t acc[4][16];
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (k < mine) ptx::tmem_ld_16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(gt & 1) * K2P_BN + (c_begin + k) * 16, acc[k]);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        if (k < mine) {
                            const int c16 = c_begin + k;
                            const uint32_t box = wrow + (c16 >> 2) * W_BOX_BYTES;
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const uint32_t addr = box + (((((c16 & 3) << 1) + h) ^ (row & 7)) << 4);
                                uint32_t x[4];
                                ptx::ld_shared_v4(addr, x[0], x[1], x[2], x[3]);
#pragma unroll
                                for (int u = 0; u < 4; ++u) {
                                    const __nv_bfloat162 old = *reinterpret_cast<__nv_bfloat162*>(&x[u]);
                                    const float lo = fmaf(-step, __uint_as_float(acc[k][h * 8 + 2 * u]), __low2float(old));
                                    const float hi = fmaf(-step, __uint_as_float(acc[k][h * 8 + 2 * u + 1]), __high2float(old));
                                    __nv_bfloat162 nw = __floats2bfloat162_rn(lo, hi);
                                    x[u] = *reinterpret_cast<uint32_t*>(&nw);
                                }
                                ptx::st_shared_v4(addr, x[0], x[1], x[2], x[3]);
                            }
                        }
                    }
                }
                ptx::tc_fence_before_sync();
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    const uint32_t ebar = ptx::smem_addr(&ctl->acc_empty[gt & 1]);
                    if (half == 0) ptx::mbar_arrive(ebar);
                    else ptx::mbar_arrive_cluster(ptx::map_to_cta(ebar, 0u));
                    ptx::mbar_arrive(ptx::smem_addr(&ctl->out_ready[s]));
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ slab generators
        // This CTA's half of the slab of A as the N x K operand: row = column of W (64 of the slab's 128), K = index j of
        // the sketch, values rounded to bf16.  Written through the generic proxy, so the arrival that tells the leader's
        // MMA thread carries a release at cluster scope when it comes from the follower.
        const int g = (int)threadIdx.x - 32 * K2P_FIXED_WARPS;
        int k = 0;
        bool ok = true;
        for (int it = cluster; it < n_items && ok; it += clusters, ++k) {
            const K2Item item = items[it];
            const PhiloxKey key = make_key(seeds.s[item.mat - seed_base]);
            const int sb = k & 1;
            ok = ptx::mbar_wait(ptx::smem_addr(&ctl->slab_empty[sb]), (((uint32_t)k >> 1) & 1u) ^ 1u, abort);
            if (!ok) break;
            k2_generate_slab<true>(slab0 + sb * slab_bytes, slab_block, kchunks, 64, item.col0 + 64 * (int)half, r, key, scale, g, 32 * K2P_GEN_WARPS);
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                const uint32_t fbar = ptx::smem_addr(&ctl->slab_full[sb]);
                if (half == 0) ptx::mbar_arrive(fbar);
                else ptx::mbar_arrive_cluster_release(ptx::map_to_cta(fbar, 0u));
            }
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                    // neither CTA leaves while the other may still arrive on its barriers or read its half of a slab
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem, tmem_cols);
    }
}

inline size_t decompress_pair_smem_bytes(int r, int slots, int cstages)
{
    const size_t kchunks = (size_t)(r + 63) / 64;
    return 2 * kchunks * 64 * 128 + (size_t)cstages * S_CHUNK_BYTES + (size_t)slots * 2 * W_BOX_BYTES + sizeof(K2PairSmem) + 1024;
}

}  // namespace flora
