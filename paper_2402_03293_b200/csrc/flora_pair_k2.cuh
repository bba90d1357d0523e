// Decompression fused with the update for ranks above 128 on CTA pairs (tcgen05.mma.cta_group::2):  W <- W - step * S A.
//
// Same structure as decompress_tc_kernel (a slab of 128 columns of A stays resident while the row tiles of W stream
// past it), with two CTAs working on one slab: an MMA multiplies the 128 rows of the sketch tile of either CTA
// (M = 256) with the slab, of which each CTA generates and holds only the 64 columns that the instruction takes
// from its shared memory (the N x K operand is split over the pair).  Half a slab is 32 KB at r = 256, so two
// buffers fit and the slab of the next item is generated while the current item streams, which a single CTA
// cannot do above r = 192 (below that the pair is faster as well, down to r = 129: measured).  The pair takes the
// row tiles of an item in turn (the leader the even ones), so an item streams in half the time and each CTA
// generates half as much per item.  Each CTA loads, combines and stores its own W tiles (two slots or more; the
// tile that will follow a tile in its slot is asked into L2 meanwhile).  The leader issues the MMAs for both, from
// two threads: a thread gets an MMA accepted only about every hundred cycles, and with sixteen of them and five
// commits per tile iteration one thread alone sets the pace of the kernel.  The two take the tile iterations in
// turn, each with two of the four accumulators and its own ring of sketch chunks, filled in step with the other's,
// and each learns from a relay thread of the follower that the follower's chunks have landed.  The combine warps,
// idle until the first accumulator is full, share the generation of the pair's first slab.
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

constexpr int K2P_FIXED_WARPS = 12;   // warp 0: W loads and stores, 1 and 7: MMA issue (leader) / relay (follower), 2-5 and 8-11: combine, 6: S loads
constexpr int K2P_GEN_WARPS = 8;      // warps 12..19: slab generators
constexpr int K2P_THREADS = 32 * (K2P_FIXED_WARPS + K2P_GEN_WARPS);
constexpr int K2P_BN = 128;           // columns of a slab (64 per CTA)
constexpr int K2P_PREFETCH_AHEAD = 0; // a W tile is asked into L2 when the tile before it in its slot is loaded (asking earlier was slower: measured)
constexpr int K2P_ACCS = 4;           // accumulators in tensor memory: two per MMA-issuing thread

struct K2PairSmem {
    uint64_t w_full[K2_MAX_SLOTS], out_ready[K2_MAX_SLOTS];
    uint64_t c_full[K2_MAX_CSTAGES], c_empty[K2_MAX_CSTAGES], acc_full[K2P_ACCS], acc_empty[K2P_ACCS], slab_full[2], slab_empty[2], slab_help;
    uint32_t tmem_base;
    int abort;
};

// A role's position in its cluster's sequence of tile iterations: item `it` (the k-th of this cluster), iteration p of n.
struct K2Cursor {
    int it, k, p, n;
    K2Item item;
};

// Cluster c (two CTAs) processes the items c, c + clusters, ...; within an item, tile iteration p covers the row tiles
// 2p (leader) and 2p + 1 (follower; it may not exist, then the follower loads and stores nothing for that iteration).
// Iterations are numbered through all items of the cluster (gt); the even ones belong to the first MMA thread, its
// ring of sketch chunks (cstages / 2 stages) and accumulators 0 and 2, the odd ones to the second.
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
    const uint32_t tmem_cols = (uint32_t)K2P_ACCS * K2P_BN;
    const int ring_stages = cstages >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < slots; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->w_full[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->out_ready[s]), 8);
        }
        for (int s = 0; s < cstages; ++s) {
            // the leader's barrier of a stage also takes the follower's word that its own chunk has landed: one wait per chunk
            ptx::mbar_init(ptx::smem_addr(&ctl->c_full[s]), half == 0 ? 2 : 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->c_empty[s]), 1);
        }
        for (int s = 0; s < K2P_ACCS; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_full[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_empty[s]), 16);                 // the eight combine warps of both CTAs (leader's barrier)
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->slab_full[s]), 2 * K2P_GEN_WARPS);  // the generator warps of both CTAs (leader's barrier)
            ptx::mbar_init(ptx::smem_addr(&ctl->slab_empty[s]), 2);                 // both MMA threads are done with the slab
        }
        ptx::mbar_init(ptx::smem_addr(&ctl->slab_help), 16);    // the combine warps of both CTAs have written their share of the first slab
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
    auto cur_load = [&](K2Cursor& c) {
        if (c.it < n_items) {
            c.item = items[c.it];
            c.n = iterations(c.item);
        }
    };
    // carries an iteration index that ran past the end of its item into the items that follow
    auto cur_norm = [&](K2Cursor& c) {
        while (c.it < n_items && c.p >= c.n) {
            c.p -= c.n;
            c.it += clusters;
            ++c.k;
            cur_load(c);
        }
    };
    auto cur_init = [&](K2Cursor& c, int first) {
        c.it = cluster;
        c.k = 0;
        c.p = first;
        c.n = 0;
        cur_load(c);
        cur_norm(c);
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ W tile loads and stores
        // One thread: the tile of iteration gt + slots goes into the slot of iteration gt as soon as the store of that one
        // has read it out, which this thread is the one to know.
        if (lane == 0) {
            K2Cursor ld, stc, pf;
            cur_init(ld, 0);
            cur_init(stc, 0);
            cur_init(pf, slots + K2P_PREFETCH_AHEAD);       // this far ahead of the loads, tiles are asked into L2: the slot's wait is then not for HBM
            RingPos pl, ps;
            int issued = 0;
            auto issue_load = [&]() {
                const TcMatrix* mat = mats + ld.item.mat;
                const int live_boxes = min(2, (mat->m - ld.item.col0 + 63) >> 6);
                const uint32_t bar = ptx::smem_addr(&ctl->w_full[pl.s]);
                if (has_tile(ld.item, ld.p)) {
                    ptx::mbar_arrive_expect_tx(bar, (uint32_t)live_boxes * W_BOX_BYTES);
                    for (int bx = 0; bx < live_boxes; ++bx)
                        ptx::tma_load_2d(w_ring + pl.s * slot_bytes + bx * W_BOX_BYTES, &mat->map_w, ld.item.col0 + bx * 64,
                                         ld.item.row0 + (2 * ld.p + (int)half) * 128, bar);
                } else {
                    ptx::mbar_arrive(bar);
                }
                ++ld.p;
                cur_norm(ld);
                pl.advance(slots);
                ++issued;
                if (pf.it < n_items) {
                    if (has_tile(pf.item, pf.p)) {
                        const TcMatrix* pmat = mats + pf.item.mat;
                        const int pboxes = min(2, (pmat->m - pf.item.col0 + 63) >> 6);
                        for (int bx = 0; bx < pboxes; ++bx)
                            ptx::tma_prefetch_l2_2d(&pmat->map_w, pf.item.col0 + bx * 64, pf.item.row0 + (2 * pf.p + (int)half) * 128);
                    }
                    ++pf.p;
                    cur_norm(pf);
                }
            };
            for (int i = 0; i < slots && ld.it < n_items; ++i) issue_load();
            bool ok = true;
            while (stc.it < n_items) {
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->out_ready[ps.s]), ps.wraps & 1u, abort);
                if (!ok) break;
                if (has_tile(stc.item, stc.p)) {
                    const TcMatrix* mat = mats + stc.item.mat;
                    const int live_boxes = min(2, (mat->m - stc.item.col0 + 63) >> 6);
                    for (int bx = 0; bx < live_boxes; ++bx)
                        ptx::tma_store_2d(&mat->map_w, stc.item.col0 + bx * 64, stc.item.row0 + (2 * stc.p + (int)half) * 128,
                                          w_ring + ps.s * slot_bytes + bx * W_BOX_BYTES);
                    ptx::tma_store_commit();
                    ptx::tma_store_wait_read<0>();          // the slot has been read out: it can be refilled
                }
                ++stc.p;
                cur_norm(stc);
                ps.advance(slots);
                if (ld.it < n_items) issue_load();
            }
            ptx::tma_store_wait_all<0>();
            if (*abort)   // loads that nobody consumed: wait (bounded) until they have landed
                for (int g = max(0, issued - slots); g < issued; ++g) ptx::mbar_wait(ptx::smem_addr(&ctl->w_full[g % slots]), (uint32_t)(g / slots) & 1u, abort);
        }
    } else if (warp == 6) {
        // ------------------------------------------------------------------ S chunk loads (bf16 copy, 64 values of the rank each)
        if (lane == 0) {
            // the chunks of an even and of the following odd iteration in turn, each into its thread's ring, so that both
            // MMA threads always have chunks to work on
            K2Cursor cs[2];
            cur_init(cs[0], 0);
            cur_init(cs[1], 1);
            RingPos prs[2];
            bool ok = true;
            // the bf16 copy of the sketches is written by the kernel before this one, which lets this one start early
            // (programmatic dependent launch): nothing else here reads what that kernel writes
            ptx::grid_dependency_wait();
            while (ok && (cs[0].it < n_items || cs[1].it < n_items)) {
                for (int kc = 0; kc < kchunks && ok; ++kc) {
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        if (cs[x].it >= n_items) continue;
                        const int st = x * ring_stages + prs[x].s;
                        ok = ptx::mbar_wait(ptx::smem_addr(&ctl->c_empty[st]), (prs[x].wraps & 1u) ^ 1u, abort);
                        if (!ok) break;
                        const uint32_t bar = ptx::smem_addr(&ctl->c_full[st]);
                        if (has_tile(cs[x].item, cs[x].p)) {
                            ptx::mbar_arrive_expect_tx(bar, S_CHUNK_BYTES);
                            ptx::tma_load_2d(c_ring + st * S_CHUNK_BYTES, &mats[cs[x].item.mat].map_sb, kc * 64,
                                             cs[x].item.row0 + (2 * cs[x].p + (int)half) * 128, bar);
                        } else {
                            ptx::mbar_arrive(bar);
                        }
                        prs[x].advance(ring_stages);
                    }
                }
#pragma unroll
                for (int x = 0; x < 2; ++x) {
                    cs[x].p += 2;
                    cur_norm(cs[x]);
                }
            }
            if (*abort)
                for (int x = 0; x < 2; ++x)
                    for (int s = 0; s < ring_stages; ++s) {
                        const uint32_t fills = prs[x].wraps + (s < prs[x].s ? 1u : 0u);
                        if (fills) ptx::mbar_wait(ptx::smem_addr(&ctl->c_full[x * ring_stages + s]), (fills - 1u) & 1u, abort);
                    }
        }
    } else if (warp == 1 || warp == 7) {
        const int x = warp == 1 ? 0 : 1;                    // which of the two issuing threads (leader) or relays (follower)
        if (lane == 0 && half == 0) {
            // -------------------------------------------------------------- MMA issuers (the pair's leader)
            // A thread waits for the slab of every item it passes, also of one in which the other thread has all the
            // iterations, and commits to slab_empty when it leaves: every phase of those barriers is then seen by
            // both, in order, which waiting by parity relies on.
            const uint32_t idesc = ptx::umma_idesc_bf16_mn(256u, (uint32_t)K2P_BN);
            const uint64_t desc_ring = ptx::umma_desc_k_sw128(c_ring + (uint32_t)(x * ring_stages) * (uint32_t)S_CHUNK_BYTES);
            K2Cursor c;
            c.it = cluster;
            c.k = 0;
            c.p = x;
            c.n = 0;
            cur_load(c);
            RingPos pc;
            int gt = x;
            bool ok = true;
            while (ok && c.it < n_items) {
                const int sb = c.k & 1;
                const uint64_t desc_slab = ptx::umma_desc_k_sw128(slab0 + sb * slab_bytes);
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->slab_full[sb]), (uint32_t)(c.k >> 1) & 1u, abort);     // both halves of the slab are written
                if (c.k == 0 && ok) ok = ptx::mbar_wait(ptx::smem_addr(&ctl->slab_help), 0u, abort);              // ... the combine warps' share of the first one too
                for (; c.p < c.n && ok; c.p += 2, gt += 2) {
                    const int a = gt & (K2P_ACCS - 1);
                    const uint32_t acc_addr = tmem + (uint32_t)a * K2P_BN;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_empty[a]), (((uint32_t)gt >> 2) & 1u) ^ 1u, abort);
                    for (int kc = 0; kc < kchunks && ok; ++kc, pc.advance(ring_stages)) {
                        const int s = pc.s;
                        const uint32_t full = ptx::smem_addr(&ctl->c_full[x * ring_stages + s]);
                        ok = ptx::mbar_wait(full, pc.wraps & 1u, abort);
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
                        ptx::umma_commit_pair(ptx::smem_addr(&ctl->c_empty[x * ring_stages + s]), (uint16_t)3u);
                    }
                    if (ok) ptx::umma_commit_pair(ptx::smem_addr(&ctl->acc_full[a]), (uint16_t)3u);
                }
                if (ok) ptx::umma_commit_pair(ptx::smem_addr(&ctl->slab_empty[sb]), (uint16_t)3u);   // every MMA of this thread that reads the slab has completed
                c.p -= c.n;
                c.it += clusters;
                ++c.k;
                cur_load(c);
            }
        } else if (lane == 0) {
            // -------------------------------------------------------------- relays (the follower): a sketch chunk has landed
            K2Cursor c;
            cur_init(c, x);
            RingPos pc;
            bool ok = true;
            while (ok && c.it < n_items) {
                for (int kc = 0; kc < kchunks; ++kc, pc.advance(ring_stages)) {
                    const uint32_t bar = ptx::smem_addr(&ctl->c_full[x * ring_stages + pc.s]);
                    ok = ptx::mbar_wait(bar, pc.wraps & 1u, abort);
                    if (!ok) break;
                    ptx::mbar_arrive_cluster(ptx::map_to_cta(bar, 0u));
                }
                c.p += 2;
                cur_norm(c);
            }
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
        if (cluster < n_items) {
            // nothing to combine yet: write a share of the first slab alongside the generator warps
            const K2Item first = items[cluster];
            const int helper = ((warp >= 8 ? warp - 4 : warp - 2) << 5) + lane;           // 0 .. 255
            if (first.tiles > 0)
                k2_generate_slab<true>(slab0, slab_block, kchunks, 64, first.col0 + 64 * (int)half, r, make_key(seeds.s[first.mat - seed_base]), scale,
                                       32 * K2P_GEN_WARPS + helper, 32 * (K2P_GEN_WARPS + 8));
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                const uint32_t hbar = ptx::smem_addr(&ctl->slab_help);
                if (half == 0) ptx::mbar_arrive(hbar);
                else ptx::mbar_arrive_cluster_release(ptx::map_to_cta(hbar, 0u));
            }
        }
        for (int it = cluster; it < n_items && ok; it += clusters) {
            const K2Item item = items[it];
            const int live_chunks = min(2, (mats[item.mat].m - item.col0 + 63) >> 6) << 2;     // 16-column chunks that hold columns of W
            const int c_begin = side * 4;
            const int mine = max(0, min(4, live_chunks - c_begin));
            for (int p = 0; p < iterations(item); ++p, ++gt, pw.advance(slots)) {
                const int s = pw.s;
                const int a = gt & (K2P_ACCS - 1);
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_full[a]), ((uint32_t)gt >> 2) & 1u, abort) &&
                     ptx::mbar_wait(ptx::smem_addr(&ctl->w_full[s]), pw.wraps & 1u, abort);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                if (has_tile(item, p)) {
                    const uint32_t wrow = w_ring + s * slot_bytes + row * 128;
                    uint32_t acc[4][16];
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (k < mine) ptx::tmem_ld_16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)a * K2P_BN + (c_begin + k) * 16, acc[k]);
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
                    const uint32_t ebar = ptx::smem_addr(&ctl->acc_empty[a]);
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
            if (item.tiles > 0)         // (an empty item pads a CTA's list: its slab is never read)
                k2_generate_slab<true>(slab0 + sb * slab_bytes, slab_block, kchunks, 64, item.col0 + 64 * (int)half, r, key, scale, g,
                                       k == 0 ? 32 * (K2P_GEN_WARPS + 8) : 32 * K2P_GEN_WARPS);      // the first slab is shared with the combine warps
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
