// Compression for ranks above 64 on CTA pairs (sm_100a: tcgen05.mma.cta_group::2):  S <- b S + a G A^T.
//
// At these ranks the r x 64 tile of A that one 64-column step needs is expensive on three counts: it must be
// generated (Philox + Box-Muller on the plain ALUs), it must sit in shared memory, and the tensor core reads it
// from there once per MMA.  All three costs are shared here:
//   * a cluster of S CTAs (S/2 pairs) streams neighbouring rows of one matrix over the same columns; every CTA
//     generates 1/S of each tile and forwards its slice to the CTAs that hold the same half of the tile
//     (bulk shared -> shared-cluster copies, no multicast loads);
//   * the two CTAs of a pair issue their MMAs together (M = 256: 128 rows of G from each CTA, N = all r columns),
//     and each holds only one half of the A tile: the instruction takes the halves of the N x K operand from
//     the two CTAs' shared memories.
// The kernel is persistent: a cluster walks a list of work units (matrix, row group, range of 64-column steps)
// that the host balanced over the clusters that can be resident; loads and generation of the next unit run
// ahead while the accumulators of the current one are written out.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "flora_ptx.cuh"
#include "flora_rng.cuh"
#include "flora_tc.cuh"

namespace flora {

constexpr int PAIR_T = 2;                   // 128-row tiles per CTA (accumulators: PAIR_T x N <= 512 tensor-memory columns)
constexpr int PAIR_FIXED_WARPS = 4;         // single-thread roles on warps 0, 4, 8, 12: G loads; MMA issue (tile 0); slice forwarding;
                                            // MMA issue (tile 1) in the leader, relay of the step's readiness in the follower
constexpr int PAIR_EPI_WARPS = 8;           // two groups of four: group t writes out tile t; between two units they generate too
constexpr int PAIR_MAX_GEN_WARPS = 16;
constexpr int PAIR_MAX_THREADS = 32 * (PAIR_FIXED_WARPS + PAIR_MAX_GEN_WARPS + PAIR_EPI_WARPS);
constexpr int PAIR_RELAY_DEPTH = 8;         // ring of the leader's per-step "operands ready" barriers (deeper than either tile ring)
inline int pair_threads(int gen_warps) { return 32 * (PAIR_FIXED_WARPS + gen_warps + PAIR_EPI_WARPS); }

struct PairSmem {
    uint64_t full_g[8], empty_g[8], full_a[8], slice_ready[8], empty_a[8], ready[PAIR_RELAY_DEPTH], acc_full, acc_empty;
    uint32_t tmem_base;
    int abort;
    int epi_go[2];
    int next_item;      // generation work items handed out so far (one item = 32 tasks of one step's slice)
    int total_steps;    // 64-column steps of all units of this cluster
};
// full_g / full_a: in the follower, its G tiles / its half of an A tile have landed (its relay watches them); in the
// leader the same arrivals and bytes go to ready[step % PAIR_RELAY_DEPTH], which the follower's relay completes.

// N: columns of the accumulators = r rounded up to a multiple of 64 (rows r .. N of A are zero).
// A CTA of rank q in its cluster belongs to pair q / 2 and holds half h = q % 2 of every A tile: rows
// [h N/2, (h+1) N/2).  Of that half it generates the rows [pair * N/S, (pair+1) * N/S) and receives the rest from
// the CTAs of the same parity.  The even CTA of a pair (the leader) issues the MMAs for both.
__global__ void __launch_bounds__(PAIR_MAX_THREADS, 1)
compress_pair_kernel(const TcMatrix* __restrict__ mats, const K1Item* __restrict__ items, const int* __restrict__ slot_begin,
                     const __grid_constant__ SeedTable seeds, int seed_base, int r, int N, float scale, float a, float b, int gstages,
                     int astages, int S, int GW, int late_wait)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    const uint32_t g_bytes = (uint32_t)PAIR_T * G_TILE_BYTES;          // one stage of the G ring
    const uint32_t a_bytes = (uint32_t)(N >> 1) * 128u;                // one stage of the A ring: this CTA's half of a tile
    const uint32_t a_ring = smem_base + (uint32_t)gstages * g_bytes;
    const uint32_t staging = a_ring + (uint32_t)astages * a_bytes;     // two 16 KB buffers, one per epilogue group
    PairSmem* ctl = reinterpret_cast<PairSmem*>(smem_raw + (staging - ptx::smem_addr(smem_raw)) + 2 * (size_t)S_CHUNK_BYTES_K1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Roles.  A warp is served by the scheduler warp % 4 of the SM.  The four single-thread roles (warps 0, 4, 8, 12)
    // share one scheduler, which gets only three of the 24 worker warps: the thread that issues the MMAs is on the
    // critical path of every step and must not queue for issue slots behind warps that saturate the ALUs.
    const int role = ((warp & 3) == 0 && warp < 4 * PAIR_FIXED_WARPS) ? (warp >> 2) : -1;    // 0: G loads, 1: MMA issue, 2: forwarder, 3: relay
    const int ww = warp < 4 * PAIR_FIXED_WARPS ? warp - (warp >> 2) - 1 : warp - PAIR_FIXED_WARPS;   // worker index, 0 .. GW + PAIR_EPI_WARPS - 1
    const uint32_t rank = ptx::cluster_ctarank();
    const uint32_t half = rank & 1u, pair = rank >> 1;
    const int pairs = S >> 1;
    const int slot = (int)(blockIdx.x / (unsigned)S);
    const int u_begin = slot_begin[slot], u_end = slot_begin[slot + 1];   // tables are written at set creation, not by kernels
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < PAIR_T * N) tmem_cols <<= 1;

    ptx::grid_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < gstages; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->full_g[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->empty_g[s]), 2);                    // both MMA issuers of the pair have consumed the G tiles
        }
        for (int s = 0; s < astages; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->full_a[s]), 1);                     // the forwarder's arrival + the peers' bytes
            ptx::mbar_init(ptx::smem_addr(&ctl->slice_ready[s]), (uint32_t)((N / S * 8 + 31) >> 5));   // one arrival per work item of the step
            ptx::mbar_init(ptx::smem_addr(&ctl->empty_a[s]), 2 * pairs);            // both MMA issuers of every pair of the cluster have consumed the tile
        }
        // leaders: one barrier per step for all that the step's MMAs need: this CTA's G tiles (the producer's arrival and
        // their bytes), its half of the A tile (the forwarder's arrival and the peers' bytes) and the follower's word
        // that its own tiles are in place
        for (int s = 0; s < PAIR_RELAY_DEPTH; ++s) ptx::mbar_init(ptx::smem_addr(&ctl->ready[s]), 3);
        ptx::mbar_init(ptx::smem_addr(&ctl->acc_full), 2);
        ptx::mbar_init(ptx::smem_addr(&ctl->acc_empty), 2 * PAIR_EPI_WARPS);        // the epilogue warps of both CTAs of the pair
        ctl->abort = 0;
        ctl->epi_go[0] = ctl->epi_go[1] = 0;
        ctl->next_item = 0;
        int steps = 0;
        for (int u = u_begin; u < u_end; ++u) steps += items[(size_t)u * S + rank].ksteps;
        ctl->total_steps = steps;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
    }
    if (role == 1) {
        ptx::tmem_alloc_pair(ptx::smem_addr(&ctl->tmem_base), tmem_cols);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                    // every CTA's barriers exist before anyone arrives on them remotely
    ptx::tc_fence_after_sync();
    // everything above touched only shared and tensor memory; G and S may have been written by the previous kernel
    // of the stream.  `late_wait`: that kernel is this library's own pre-scaling of S, which does not touch G.
    if (!late_wait) ptx::grid_dependency_wait();
    const uint32_t tmem = ctl->tmem_base;
    volatile int* abort = &ctl->abort;

    if (role == 0) {
        // ------------------------------------------------------------------ TMA producer: this CTA's rows of G
        if (lane == 0) {
            int g = 0, issued = 0;
            RingPos pg, pp;
            bool ok = true;
            for (int u = u_begin; u < u_end && ok; ++u) {
                const K1Item item = items[(size_t)u * S + rank];
                const TcMatrix* mat = mats + item.mat;
                if (item.tiles > 0) ptx::prefetch_tensormap(&mat->map_g);
                for (int ks = 0; ks < item.ksteps; ++ks, ++g, pg.advance(gstages), pp.advance(PAIR_RELAY_DEPTH)) {
                    const int s = pg.s;
                    ok = ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->empty_g[s]), (pg.wraps & 1u) ^ 1u, abort);
                    if (!ok) break;
                    // a leader's loads complete on the step's barrier, a follower's on its own (its relay watches that one)
                    const uint32_t bar = half == 0 ? ptx::smem_addr(&ctl->ready[pp.s]) : ptx::smem_addr(&ctl->full_g[s]);
                    if (item.tiles > 0) {
                        ptx::mbar_arrive_expect_tx(bar, (uint32_t)item.tiles * G_TILE_BYTES);
                        for (int t = 0; t < item.tiles; ++t)
                            ptx::tma_load_2d(smem_base + s * g_bytes + t * G_TILE_BYTES, &mat->map_g, (item.kstep0 + ks) * 64, item.row0 + t * 128, bar);
                    } else {
                        ptx::mbar_arrive(bar);                                   // a CTA without rows loads nothing
                    }
                    issued = g + 1;
                }
            }
            if (*abort && half == 1) {
                // nobody consumes any more: wait (bounded) until the copies still in flight have landed (a leader's loads
                // complete on barriers that also need the forwarder and the follower; after an abort the kernel's final
                // cluster-wide barrier comes long after the two microseconds a load takes)
                for (int k = max(0, issued - gstages); k < issued; ++k)
                    ptx::mbar_wait(ptx::smem_addr(&ctl->full_g[k % gstages]), (uint32_t)(k / gstages) & 1u, abort);
            }
        }
    } else if (role == 1 || (role == 3 && half == 0)) {
        // ------------------------------------------------------------------ MMA issuers (the pair's leader only)
        // Two threads in two warps, one per 128-row tile: a thread gets an MMA accepted only every 120 cycles or so
        // whatever its size, and between the MMAs of two steps come its waits and commits, so one thread alone leaves
        // the tensor core idle a third of the time.  Each commits its own MMAs to the barriers that release a stage;
        // those barriers count both.  (The follower's warp of role 1 has nothing to do; its warp of role 3 is the relay.)
        if (lane == 0 && half == 0) {
            const int ti = role == 1 ? 0 : 1;
            const uint32_t idesc = ptx::umma_idesc_bf16_mn(256u, (uint32_t)N);
            const uint64_t desc_base = ptx::umma_desc_k_sw128(smem_base);
            const uint16_t mask_pair = (uint16_t)(3u << rank), mask_all = (uint16_t)((1u << S) - 1u);
            int g = 0, done = 0;
            RingPos pg, pa, pp;
            bool ok = true;
            for (int u = u_begin; u < u_end && ok; ++u, ++done) {
                const K1Item item = items[(size_t)u * S + rank];
                const int pair_tiles = max(item.tiles, items[(size_t)u * S + rank + 1].tiles);
                // the accumulators of the previous unit have been read out by both CTAs
                if (done > 0) ok = ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->acc_empty), (uint32_t)(done - 1) & 1u, abort);
                for (int ks = 0; ks < item.ksteps && ok; ++ks, ++g, pg.advance(gstages), pa.advance(astages), pp.advance(PAIR_RELAY_DEPTH)) {
                    const int sg = pg.s, sa = pa.s, sp = pp.s;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->ready[sp]), pp.wraps & 1u, abort);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t ebar_g = ptx::smem_addr(&ctl->empty_g[sg]), ebar_a = ptx::smem_addr(&ctl->empty_a[sa]);
                    if (pair_tiles > 0) {
                        // descriptors differ from the ring base only in the start-address field (16-byte units); the same
                        // offsets address the follower's copy of the rings
                        const uint64_t dstage = desc_base + (uint64_t)((sg * g_bytes) >> 4);
                        const uint64_t da_tile = desc_base + (uint64_t)((a_ring - smem_base + sa * a_bytes) >> 4);
                        if (ti < pair_tiles) {
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk)
                                ptx::umma_bf16_pair(tmem + ti * N, dstage + (uint64_t)((ti * G_TILE_BYTES + kk * 32) >> 4), da_tile + (uint64_t)(kk * 2), idesc,
                                                    (ks | kk) != 0);
                        }
                        ptx::umma_commit_pair(ebar_g, mask_pair);
                        ptx::umma_commit_pair(ebar_a, mask_all);
                    } else {
                        // a pair without rows consumes nothing, but keeps the rings' bookkeeping in step
                        ptx::mbar_arrive(ebar_g);
                        ptx::mbar_arrive_cluster(ptx::map_to_cta(ebar_g, rank + 1));
                        for (int d = 0; d < S; ++d) ptx::mbar_arrive_cluster(ptx::map_to_cta(ebar_a, d));
                    }
                }
                if (!ok) break;
                const uint32_t fbar = ptx::smem_addr(&ctl->acc_full);
                if (pair_tiles > 0) {
                    ptx::umma_commit_pair(fbar, mask_pair);
                } else {
                    ptx::mbar_arrive(fbar);
                    ptx::mbar_arrive_cluster(ptx::map_to_cta(fbar, rank + 1));
                }
            }
        }
    } else if (role == 2) {
        // ------------------------------------------------------------------ forwarder: this CTA's slice of A to the CTAs of the same parity
        if (lane == 0) {
            const uint32_t slice_bytes = (uint32_t)(N / S) * 128u;
            int g = 0;
            RingPos pa, pp;
            bool ok = true;
            for (int u = u_begin; u < u_end && ok; ++u) {
                const int ksteps = items[(size_t)u * S + rank].ksteps;
                for (int ks = 0; ks < ksteps; ++ks, ++g, pa.advance(astages), pp.advance(PAIR_RELAY_DEPTH)) {
                    const int s = pa.s;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->slice_ready[s]), pa.wraps & 1u, abort);
                    if (!ok) break;
                    // the same barrier offset in every CTA of this parity: the step's barrier among leaders, the A stage's among followers
                    const uint32_t fbar = half == 0 ? ptx::smem_addr(&ctl->ready[pp.s]) : ptx::smem_addr(&ctl->full_a[s]);
                    if (pairs > 1) {
                        const uint32_t src = a_ring + s * a_bytes + pair * slice_bytes;
                        ptx::mbar_arrive_expect_tx(fbar, (uint32_t)(pairs - 1) * slice_bytes);   // own slice is in place; the peers' bytes to come
                        for (int d = 0; d < pairs; ++d)
                            if (d != (int)pair) ptx::bulk_copy_to_peer(ptx::map_to_cta(src, 2u * d + half), src, slice_bytes, ptx::map_to_cta(fbar, 2u * d + half));
                    } else {
                        ptx::mbar_arrive(fbar);
                    }
                }
            }
        }
    } else if (role == 3) {
        // ------------------------------------------------------------------ relay (follower only; the leader's warp issues MMAs, above): tells the leader that this CTA's
        // G tiles and half of the A tile of a step are in place
        if (lane == 0 && half == 1) {
            int g = 0;
            RingPos pg, pa, pp;
            bool ok = true;
            for (int u = u_begin; u < u_end && ok; ++u) {
                const int ksteps = items[(size_t)u * S + rank].ksteps;
                for (int ks = 0; ks < ksteps; ++ks, ++g, pg.advance(gstages), pa.advance(astages), pp.advance(PAIR_RELAY_DEPTH)) {
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->full_g[pg.s]), pg.wraps & 1u, abort) &&
                         ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->full_a[pa.s]), pa.wraps & 1u, abort);
                    if (!ok) break;
                    ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_addr(&ctl->ready[pp.s]), rank - 1));
                }
            }
        } else if (lane == 0) {
            // the leader's own relay ring is fed by the follower; nothing to do here
        }
    } else {
        // ------------------------------------------------------------------ workers: generation of A, and the epilogue
        // The slice of one step is cut into work items of 32 tasks (a task: one row of A x one 16-byte chunk = eight
        // values, a long dependent chain of integer and floating-point operations).  Every worker warp claims the next
        // item from a counter in shared memory, so as many slices are in the making at once as there are free stages
        // and idle warps: it is the latency of a task, not the issue rate, that bounds one slice.  The last
        // PAIR_EPI_WARPS workers also write the accumulators out: they claim no item of a unit later than the one
        // whose accumulators they have to write next, so the MMA issuer never waits for them behind work it must
        // itself release.
        const bool epi_duty = ww >= GW;
        const int rows_per_cta = N / S;
        const int my_tasks = rows_per_cta * 8;                    // (row, 16-byte chunk) pairs of this CTA's slice
        const int parts = (my_tasks + 31) >> 5;                   // work items per step
        const int lrow0 = (int)pair * rows_per_cta;               // first row of the slice inside this CTA's half
        const int j0 = (int)half * (N >> 1) + lrow0;              // the same row counted in A
        const int total_items = ctl->total_steps * parts;
        // cursor over the units: the unit that holds step g (claims only move forward)
        int cu = u_begin, cu_g0 = 0, cu_steps = 0, cu_kstep0 = 0;
        PhiloxKey key = make_key(0);
        auto load_cursor = [&]() {
            if (cu < u_end) {
                const K1Item it = items[(size_t)cu * S + rank];
                cu_steps = it.ksteps;
                cu_kstep0 = it.kstep0;
                key = make_key(seeds.s[it.mat - seed_base]);
            } else {
                cu_steps = 1 << 30;
            }
        };
        load_cursor();
        auto seek = [&](int g) {
            while (g >= cu_g0 + cu_steps) {
                cu_g0 += cu_steps;
                ++cu;
                load_cursor();
            }
        };
        bool ok = true;
        auto generate = [&](int w) {
            const int g = w / parts, part = w - g * parts;
            seek(g);
            const int s = g % astages;
            ok = ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->empty_a[s]), ((uint32_t)(g / astages) & 1u) ^ 1u, abort);
            if (!ok) return;
            const uint32_t a_tile = a_ring + s * a_bytes;
            const uint32_t q0 = (uint32_t)(cu_kstep0 + (g - cu_g0)) * 16u;
            const int t = part * 32 + lane;
            if (t < my_tasks) {
                const int lr = lrow0 + (t >> 3), j = j0 + (t >> 3), c = t & 7;
                uint2 lo = make_uint2(0u, 0u), hi = make_uint2(0u, 0u);
                if (j < r) {
                    lo = projection_quad_bf16(q0 + 2 * c, (uint32_t)j, key, scale);
                    hi = projection_quad_bf16(q0 + 2 * c + 1, (uint32_t)j, key, scale);
                }
                ptx::st_shared_v4(a_tile + lr * 128 + ((c ^ (lr & 7)) << 4), lo.x, lo.y, hi.x, hi.y);
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->slice_ready[s]));
        };

        if (!epi_duty) {
            while (ok) {
                int w = 0;
                if (lane == 0) w = atomicAdd(&ctl->next_item, 1);
                w = __shfl_sync(0xffffffffu, w, 0);
                if (w >= total_items) break;
                generate(w);
            }
        } else {
            // Epilogue: group t writes out tile t of every unit.  Warp w of a group owns tensor-memory lanes
            // 32*(w%4) .. +31, i.e. those rows of the tile.  The accumulator leaves in chunks of 32 columns x 128 rows
            // (16 KB): registers -> the group's staging buffer in the 128-byte-swizzled layout of the sketch's tensor map
            // -> one bulk tensor operation, clipped by the hardware at the sketch's last row and column:
            //   add   S <- S + a*acc   (b == 1, or several units share the rows and S was scaled by b beforehand):
            //         a bulk reduction, nothing is read back;
            //   store S <- a*acc       (b == 0 and the unit owns its rows);
            //   rmw   S <- b*S + a*acc (the unit owns its rows): each thread reads its row's old values straight from
            //         global memory.
            const int ew = ww - GW;
            const int grp = ew >> 2;
            const int quarter = warp & 3;
            const bool leader = (ew & 3) == 0 && lane == 0;
            const int trow = quarter * 32 + lane;                     // row inside a tile
            const uint32_t bar_a = 1u + 2u * (uint32_t)grp, bar_b = bar_a + 1u;
            const uint32_t buf = staging + (uint32_t)grp * S_CHUNK_BYTES_K1;
            const uint32_t brow = buf + (uint32_t)trow * 128u;
            const int nchunks = (r + 31) >> 5;
            bool waited = !late_wait, eok = true;
            for (int u = u_begin, done = 0; u < u_end; ++u, ++done) {
                // until the accumulators of unit u are due, help with the generation of units up to u
                while (ok) {
                    int w = 0, mine = 0;
                    if (lane == 0) {
                        w = *(volatile int*)&ctl->next_item;
                        if (w < total_items) {
                            seek(w / parts);
                            if (cu <= u) mine = atomicCAS(&ctl->next_item, w, w + 1) == w ? 1 : 2;    // 2: somebody else took it, look again
                        }
                    }
                    mine = __shfl_sync(0xffffffffu, mine, 0);
                    if (mine == 0) break;
                    if (mine == 2) continue;
                    w = __shfl_sync(0xffffffffu, w, 0);
                    generate(w);
                }
                const K1Item item = items[(size_t)u * S + rank];
                const TcMatrix* mat = mats + item.mat;
                if (eok) eok = ok && ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->acc_full), (uint32_t)done & 1u, abort);
                ptx::tc_fence_after_sync();
                if (!waited) {
                    ptx::grid_dependency_wait();
                    waited = true;
                }
                if (grp < item.tiles) {
                    const bool add = item.direct == 0 || b == 1.0f;
                    const bool rmw = !add && b != 0.0f;
                    const int row = item.row0 + grp * 128 + trow;
                    const float* old_row = mat->S + (int64_t)row * mat->lds;
                    const bool row_ok = row < mat->n;
                    for (int c = 0; c < nchunks; ++c) {
                        if (leader) {
                            const bool go = eok && !*abort;
                            if (go) ptx::tma_store_wait_read<0>();    // the previous chunk has been read out of the staging buffer
                            ctl->epi_go[grp] = go ? 1 : 0;
                        }
                        ptx::named_barrier_sync(bar_a, 128);
                        if (!*(volatile int*)&ctl->epi_go[grp]) break;      // uniform: written before the barrier by one thread
#pragma unroll
                        for (int hc = 0; hc < 2; ++hc) {
                            const int col0 = c * 32 + hc * 16;
                            float o[16];
                            if (rmw) {
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    const int col = col0 + 4 * q;
                                    if (row_ok && col + 3 < r) {
                                        const float4 v4 = *reinterpret_cast<const float4*>(old_row + col);
                                        o[4 * q] = v4.x; o[4 * q + 1] = v4.y; o[4 * q + 2] = v4.z; o[4 * q + 3] = v4.w;
                                    } else {
#pragma unroll
                                        for (int e = 0; e < 4; ++e) o[4 * q + e] = (row_ok && col + e < r) ? old_row[col + e] : 0.0f;
                                    }
                                }
                            }
                            uint32_t v[16];
                            if (col0 < N) {
                                ptx::tmem_ld_16(tmem + ((uint32_t)(quarter * 32) << 16) + grp * N + col0, v);
                                ptx::tmem_ld_wait();
                            } else {
#pragma unroll
                                for (int k = 0; k < 16; ++k) v[k] = 0u;
                            }
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const uint32_t addr = brow + (uint32_t)(((hc * 4 + q) ^ (trow & 7)) << 4);
                                float x0 = a * __uint_as_float(v[4 * q]), x1 = a * __uint_as_float(v[4 * q + 1]);
                                float x2 = a * __uint_as_float(v[4 * q + 2]), x3 = a * __uint_as_float(v[4 * q + 3]);
                                if (rmw) {
                                    x0 = fmaf(b, o[4 * q], x0);
                                    x1 = fmaf(b, o[4 * q + 1], x1);
                                    x2 = fmaf(b, o[4 * q + 2], x2);
                                    x3 = fmaf(b, o[4 * q + 3], x3);
                                }
                                ptx::st_shared_v4(addr, __float_as_uint(x0), __float_as_uint(x1), __float_as_uint(x2), __float_as_uint(x3));
                            }
                        }
                        ptx::fence_proxy_async_smem();
                        ptx::named_barrier_sync(bar_b, 128);
                        if (leader && !*abort) {
                            if (add) ptx::tma_reduce_add_2d(&mat->map_s, c * 32, item.row0 + grp * 128, buf);
                            else ptx::tma_store_2d(&mat->map_s, c * 32, item.row0 + grp * 128, buf);
                            ptx::tma_store_commit();
                        }
                    }
                }
                // this warp has read all it needs from the accumulators of this unit: tell the pair's MMA issuer
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    const uint32_t ebar = ptx::smem_addr(&ctl->acc_empty);
                    if (half == 0) ptx::mbar_arrive(ebar);
                    else ptx::mbar_arrive_cluster(ptx::map_to_cta(ebar, rank - 1));
                }
            }
            if (leader) ptx::tma_store_wait_all<0>();                 // the sketches are complete in global memory before the CTA ends
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                    // no CTA leaves while peers may still store into it or arrive on its barriers
    if (role == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem, tmem_cols);
    }
}

}  // namespace flora
