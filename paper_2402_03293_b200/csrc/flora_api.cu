// C ABI of the Flora hot path (see include/flora.h for the contract of every entry point).
// This file validates arguments, picks a kernel family and launches; all arithmetic of the path
// lives in the kernels of flora_simt.cuh (fp32 SIMT), flora_tc.cuh (tcgen05 tensor cores; host side in flora_tc_host.cuh)
// and flora_gram.cuh (momentum transfer).
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/flora.h"
#include "flora_rng.cuh"
#include "flora_simt.cuh"
#include "flora_pool.cuh"
#include "flora_tc_host.cuh"
#include "flora_gram.cuh"

using namespace flora;

namespace {

std::atomic<uint64_t> g_launches{0};
std::atomic<int> g_force_path{0};

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
inline flora_status launched()
{
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaPeekAtLastError() == cudaSuccess ? FLORA_OK : FLORA_ERR_CUDA;
}
inline float projection_scale(int r) { return 1.0f / sqrtf((float)r); }
inline size_t elem_size(int32_t dt) { return dt == FLORA_BF16 ? 2 : 4; }

flora_status check_mat(const flora_mat* a, bool f32_only)
{
    if (!a) return FLORA_ERR_NULL;
    if (a->dtype != FLORA_F32 && a->dtype != FLORA_BF16) return FLORA_ERR_DTYPE;
    if (f32_only && a->dtype != FLORA_F32) return FLORA_ERR_DTYPE;
    if (a->rows < 0 || a->cols < 0 || a->ld < a->cols) return FLORA_ERR_SHAPE;
    if (a->rows > 0 && a->cols > 0) {
        if (!a->data) return FLORA_ERR_NULL;
        if (reinterpret_cast<uintptr_t>(a->data) % elem_size(a->dtype)) return FLORA_ERR_ALIGN;
    }
    return FLORA_OK;
}

// G (or W) against its sketch: same row count, rank in range.
flora_status check_pair(const flora_mat* big, const flora_mat* sketch)
{
    flora_status st = check_mat(big, false);
    if (st) return st;
    st = check_mat(sketch, true);
    if (st) return st;
    if (sketch->cols < 1 || sketch->cols > 256) return FLORA_ERR_RANK;
    if (sketch->rows != big->rows) return FLORA_ERR_SHAPE;
    if (big->cols > (int64_t)4 * 0x7FFFFFFF || big->rows > 0x7FFFFFFFll * 32) return FLORA_ERR_UNSUPPORTED;
    return FLORA_OK;
}

// ------------------------------------------------------------------------------------------------
// SIMT launches
// ------------------------------------------------------------------------------------------------
flora_status simt_compress(const flora_mat* G, flora_mat* S, uint64_t seed, float a, float b, cudaStream_t st)
{
    const int r = (int)S->cols;
    if (G->rows == 0) return FLORA_OK;
    const unsigned grid = (unsigned)((G->rows + 31) / 32);
    if (G->dtype == FLORA_BF16)
        simt_compress_kernel<__nv_bfloat16><<<grid, SIMT_THREADS, 0, st>>>(
            (const __nv_bfloat16*)G->data, G->rows, G->cols, G->ld, (float*)S->data, S->ld, r, make_key(seed),
            projection_scale(r), a, b);
    else
        simt_compress_kernel<float><<<grid, SIMT_THREADS, 0, st>>>(
            (const float*)G->data, G->rows, G->cols, G->ld, (float*)S->data, S->ld, r, make_key(seed),
            projection_scale(r), a, b);
    return launched();
}

flora_status simt_decompress(flora_mat* W, const flora_mat* C, uint64_t seed, float step, cudaStream_t st)
{
    const int r = (int)C->cols;
    if (W->rows == 0 || W->cols == 0) return FLORA_OK;
    dim3 grid((unsigned)((W->cols + 63) / 64), (unsigned)((W->rows + 31) / 32));
    if (grid.y > 65535) return FLORA_ERR_UNSUPPORTED;
    if (W->dtype == FLORA_BF16)
        simt_decompress_kernel<__nv_bfloat16><<<grid, SIMT_THREADS, 0, st>>>(
            (__nv_bfloat16*)W->data, W->rows, W->cols, W->ld, (const float*)C->data, C->ld, r, make_key(seed),
            projection_scale(r), step);
    else
        simt_decompress_kernel<float><<<grid, SIMT_THREADS, 0, st>>>(
            (float*)W->data, W->rows, W->cols, W->ld, (const float*)C->data, C->ld, r, make_key(seed),
            projection_scale(r), step);
    return launched();
}

// T (r x r, zeroed here) <- A_old A_new^T with the SIMT kernel.
flora_status simt_gram(float* T, int r, int64_t m, int32_t operand, uint64_t s_old, uint64_t s_new, cudaStream_t st)
{
    if (cudaMemsetAsync(T, 0, sizeof(float) * r * r, st) != cudaSuccess) return FLORA_ERR_CUDA;
    if (m == 0) return FLORA_OK;
    const int tiles = (r + 31) / 32;
    int64_t splits = (m + 511) / 512;
    if (splits > 1024) splits = 1024;
    int64_t kper = ((m + splits - 1) / splits + 31) / 32 * 32;
    splits = (m + kper - 1) / kper;
    dim3 grid((unsigned)(tiles * tiles), (unsigned)splits);
    simt_gram_kernel<<<grid, SIMT_THREADS, 0, st>>>(T, r, m, kper, operand == FLORA_BF16, make_key(s_old),
                                                    make_key(s_new), projection_scale(r));
    return launched();
}

flora_status simt_apply_gram(flora_mat* dst, const flora_mat* src, const float* T, float a, float b, cudaStream_t st)
{
    if (dst->rows == 0) return FLORA_OK;
    const unsigned grid = (unsigned)((dst->rows + 7) / 8);
    simt_apply_gram_kernel<<<grid, SIMT_THREADS, 0, st>>>((float*)dst->data, dst->ld, (const float*)src->data, src->ld,
                                                          dst->rows, (int)dst->cols, T, a, b);
    return launched();
}

flora_status check_transfer(const flora_mat* dst, const flora_mat* src, int64_t m, int32_t operand)
{
    flora_status st = check_mat(dst, true);
    if (st) return st;
    st = check_mat(src, true);
    if (st) return st;
    if (operand != FLORA_F32 && operand != FLORA_BF16) return FLORA_ERR_DTYPE;
    if (dst->cols < 1 || dst->cols > 256 || src->cols != dst->cols) return FLORA_ERR_RANK;
    if (src->rows != dst->rows || m < 0 || m > (int64_t)4 * 0x7FFFFFFF) return FLORA_ERR_SHAPE;
    return FLORA_OK;
}

// dst <- b dst + a src (A_old A_new^T) with T in the given scratch (r*r floats).
flora_status transfer_with_scratch(flora_mat* dst, const flora_mat* src, int64_t m, int32_t operand, uint64_t s_old,
                                   uint64_t s_new, float a, float b, float* T, cudaStream_t st)
{
    flora_status rc = simt_gram(T, (int)dst->cols, m, operand, s_old, s_new, st);
    if (rc) return rc;
    return simt_apply_gram(dst, src, T, a, b, st);
}

// ------------------------------------------------------------------------------------------------
// Scratch for flora_resample_transfer_static: lives in the library image, one copy per GPU that loads it.
// In host code the name below is only a handle; the device address comes from cudaGetSymbolAddress.
// ------------------------------------------------------------------------------------------------
constexpr int STATIC_TRANSFER_MAX_R = 256;
static __device__ __align__(256) float g_static_transfer_scratch[STATIC_TRANSFER_MAX_R * STATIC_TRANSFER_MAX_R];

constexpr int MAX_DEVICES = 64;
std::mutex g_static_mutex;
float* g_static_scratch_addr[MAX_DEVICES] = {};

// Device address of the scratch on the current device, looked up once per device.
flora_status static_scratch_for_current_device(float** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return FLORA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_transfer_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return FLORA_ERR_CUDA;
        }
        g_static_scratch_addr[dev] = static_cast<float*>(p);
    }
    *out = g_static_scratch_addr[dev];
    return FLORA_OK;
}

bool use_tc_compress(const flora_mat* big, const flora_mat* sketch)
{
    return g_force_path.load(std::memory_order_relaxed) != 1 && tc_compress_supported(big, sketch);
}
bool use_tc_decompress(const flora_mat* big, const flora_mat* sketch)
{
    return g_force_path.load(std::memory_order_relaxed) != 1 && tc_decompress_supported(big, sketch);
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// set object
// ------------------------------------------------------------------------------------------------
struct flora_set {
    std::vector<flora_mat> G, W, S;
    int r = 0;
    bool has_G = false, has_W = false;
    TcSet tc;   // tensor-core work lists and descriptors (empty when the set is not eligible)
};

extern "C" {

flora_status flora_compress_accumulate(const flora_mat* G, flora_mat* C, uint64_t seed, int r, void* stream)
{
    flora_status st = check_pair(G, C);
    if (st) return st;
    if (r != C->cols) return FLORA_ERR_RANK;
    if (G->rows == 0 || G->cols == 0) return FLORA_OK;
    if (use_tc_compress(G, C)) return tc_compress_single(G, C, seed, 1.0f, 1.0f, as_stream(stream), g_launches);
    return simt_compress(G, C, seed, 1.0f, 1.0f, as_stream(stream));
}

flora_status flora_momentum_step(const flora_mat* G, flora_mat* M, float beta, uint64_t seed, void* stream)
{
    flora_status st = check_pair(G, M);
    if (st) return st;
    if (G->rows == 0) return FLORA_OK;
    if (G->cols > 0 && use_tc_compress(G, M)) return tc_compress_single(G, M, seed, 1.0f - beta, beta, as_stream(stream), g_launches);
    return simt_compress(G, M, seed, 1.0f - beta, beta, as_stream(stream));
}

flora_status flora_momentum_step_resampled(const flora_mat* G, flora_mat* M, float beta, uint64_t seed_old, uint64_t seed_new, void* stream)
{
    flora_status st = check_pair(G, M);
    if (st) return st;
    if (G->rows == 0) return FLORA_OK;
    // M <- beta (M A_old A_new^T): the transfer's own scaling; then M <- M + (1 - beta) G A_new^T, a pure accumulation
    st = flora_transfer_axpby(M, M, G->cols, G->dtype, seed_old, seed_new, beta, 0.0f, stream);
    if (st) return st;
    if (G->cols > 0 && use_tc_compress(G, M)) return tc_compress_single(G, M, seed_new, 1.0f - beta, 1.0f, as_stream(stream), g_launches);
    return simt_compress(G, M, seed_new, 1.0f - beta, 1.0f, as_stream(stream));
}

flora_status flora_decompress_apply(flora_mat* W, const flora_mat* C, uint64_t seed, float lr, float scale, void* stream)
{
    flora_status st = check_pair(W, C);
    if (st) return st;
    if (W->rows == 0 || W->cols == 0) return FLORA_OK;
    if (use_tc_decompress(W, C)) return tc_decompress_single(W, C, seed, lr * scale, as_stream(stream), g_launches);
    return simt_decompress(W, C, seed, lr * scale, as_stream(stream));
}

flora_status flora_transfer_axpby(flora_mat* dst, const flora_mat* src, int64_t m, int32_t operand, uint64_t seed_old,
                                  uint64_t seed_new, float a, float b, void* stream)
{
    flora_status st = check_transfer(dst, src, m, operand);
    if (st) return st;
    if (dst->rows == 0) return FLORA_OK;
    const int r = (int)dst->cols;
    if (operand == FLORA_BF16 && g_force_path.load() != 1) {
        std::vector<GramJob> jobs(1);
        jobs[0] = GramJob{nullptr, (float*)dst->data, (const float*)src->data, dst->ld, src->ld, (int32_t)dst->rows, (int32_t)m, seed_old, seed_new, 0, 0};
        if (dst->rows <= 0x7FFFFFFF && m <= 0x7FFFFFFF) return transfer_tc(jobs, r, a, b, as_stream(stream), g_launches);
    }
    float* T = nullptr;
    if (scratch_alloc((void**)&T, sizeof(float) * r * r, as_stream(stream)) != cudaSuccess) {
        cudaGetLastError();
        return FLORA_ERR_ALLOC;
    }
    st = transfer_with_scratch(dst, src, m, operand, seed_old, seed_new, a, b, T, as_stream(stream));
    if (cudaFreeAsync(T, as_stream(stream)) != cudaSuccess && st == FLORA_OK) st = FLORA_ERR_CUDA;
    return st;
}

flora_status flora_resample_transfer(flora_mat* M, int64_t m, int32_t operand, uint64_t seed_old, uint64_t seed_new, void* stream)
{
    return flora_transfer_axpby(M, M, m, operand, seed_old, seed_new, 1.0f, 0.0f, stream);
}

flora_status flora_resample_transfer_static(flora_mat* M, int64_t m, int32_t operand, uint64_t seed_old, uint64_t seed_new, void* stream)
{
    flora_status st = check_transfer(M, M, m, operand);
    if (st) return st;
    const int64_t r = M->cols;
    if (r * r > (int64_t)STATIC_TRANSFER_MAX_R * STATIC_TRANSFER_MAX_R) return FLORA_ERR_RANK;   // larger than the built-in scratch
    if (M->rows == 0) return FLORA_OK;
    float* T = nullptr;
    st = static_scratch_for_current_device(&T);
    if (st) return st;
    // T is cleared inside (it still holds the previous call's product), then filled and applied; bf16 operands take the
    // tensor-core kernels of flora_resample_transfer (one matrix needs no tables: its job travels as a kernel parameter)
    if (operand == FLORA_BF16 && g_force_path.load() != 1 && M->rows <= 0x7FFFFFFF && m <= 0x7FFFFFFF) {
        std::vector<GramJob> jobs(1);
        jobs[0] = GramJob{nullptr, (float*)M->data, (const float*)M->data, M->ld, M->ld, (int32_t)M->rows, (int32_t)m, seed_old, seed_new, 0, 0};
        return transfer_tc(jobs, (int)r, 1.0f, 0.0f, as_stream(stream), g_launches, nullptr, nullptr, T);
    }
    return transfer_with_scratch(M, M, m, operand, seed_old, seed_new, 1.0f, 0.0f, T, as_stream(stream));
}

flora_status flora_materialize_A(flora_mat* out, uint64_t seed, void* stream)
{
    flora_status st = check_mat(out, false);
    if (st) return st;
    if (out->rows < 1 || out->rows > 256) return FLORA_ERR_RANK;
    if (out->cols == 0) return FLORA_OK;
    if (out->cols > (int64_t)4 * 0x7FFFFFFF) return FLORA_ERR_UNSUPPORTED;
    const int r = (int)out->rows;
    const int64_t tasks = (out->cols + 3) / 4 * r;
    const unsigned grid = (unsigned)((tasks + 255) / 256);
    if (out->dtype == FLORA_BF16)
        materialize_kernel<__nv_bfloat16><<<grid, 256, 0, as_stream(stream)>>>((__nv_bfloat16*)out->data, r, out->cols, out->ld,
                                                                              make_key(seed), projection_scale(r));
    else
        materialize_kernel<float><<<grid, 256, 0, as_stream(stream)>>>((float*)out->data, r, out->cols, out->ld, make_key(seed),
                                                                      projection_scale(r));
    return launched();
}

// ------------------------------------------------------------------------------------------------
// sets
// ------------------------------------------------------------------------------------------------
flora_status flora_set_create(int count, const flora_mat* G, const flora_mat* W, const flora_mat* S, flora_set** out)
{
    if (!out || !S || (!G && !W)) return FLORA_ERR_NULL;
    if (count < 0) return FLORA_ERR_SHAPE;
    *out = nullptr;
    int r = count ? (int)S[0].cols : 1;
    for (int i = 0; i < count; ++i) {
        const flora_mat* big = G ? &G[i] : &W[i];
        flora_status st = check_pair(big, &S[i]);
        if (st) return st;
        if (S[i].cols != r) return FLORA_ERR_RANK;
        if (G && W) {
            st = check_pair(&W[i], &S[i]);
            if (st) return st;
            if (W[i].cols != G[i].cols) return FLORA_ERR_SHAPE;
            if (W[i].dtype != G[i].dtype) return FLORA_ERR_DTYPE;
        }
    }
    flora_set* s = new (std::nothrow) flora_set();
    if (!s) return FLORA_ERR_ALLOC;
    s->r = r;
    s->has_G = G != nullptr;
    s->has_W = W != nullptr;
    s->S.assign(S, S + count);
    if (G) s->G.assign(G, G + count);
    if (W) s->W.assign(W, W + count);
    flora_status st = tc_set_build(s->tc, s->G, s->W, s->S);
    if (st) {
        tc_set_free(s->tc);
        delete s;
        return st;
    }
    *out = s;
    return FLORA_OK;
}

flora_status flora_set_destroy(flora_set* set)
{
    if (!set) return FLORA_OK;
    tc_set_free(set->tc);
    delete set;
    return FLORA_OK;
}

flora_status flora_set_rebind_gradients(flora_set* set, const flora_mat* G, void* stream)
{
    if (!set || !G) return FLORA_ERR_NULL;
    if (!set->has_G) return FLORA_ERR_UNSUPPORTED;
    for (size_t i = 0; i < set->G.size(); ++i) {
        flora_status st = check_mat(&G[i], false);
        if (st) return st;
        if (G[i].rows != set->G[i].rows || G[i].cols != set->G[i].cols || G[i].ld != set->G[i].ld) return FLORA_ERR_SHAPE;
        if (G[i].dtype != set->G[i].dtype) return FLORA_ERR_DTYPE;
    }
    std::vector<flora_mat> newG(G, G + set->G.size());
    flora_status st = tc_set_rebind(set->tc, newG, as_stream(stream));
    if (st) return st;
    set->G.swap(newG);
    return FLORA_OK;
}

// behind_own_transfer: the kernel before this call on the stream is the library's own transfer, which does not touch G
static flora_status set_compress(flora_set* set, const uint64_t* seeds, float a, float b, void* stream, bool behind_own_transfer = false)
{
    if (!set || !seeds) return FLORA_ERR_NULL;
    if (!set->has_G) return FLORA_ERR_UNSUPPORTED;
    if (set->tc.compress_ready && g_force_path.load() != 1)
        return tc_set_compress(set->tc, seeds, a, b, as_stream(stream), g_launches, behind_own_transfer);
    for (size_t i = 0; i < set->G.size(); ++i) {
        if (set->G[i].rows == 0) continue;
        flora_status st = simt_compress(&set->G[i], &set->S[i], seeds[i], a, b, as_stream(stream));
        if (st) return st;
    }
    return FLORA_OK;
}

flora_status flora_set_compress_accumulate(flora_set* set, const uint64_t* seeds, void* stream)
{
    return set_compress(set, seeds, 1.0f, 1.0f, stream);
}

flora_status flora_set_momentum_step(flora_set* set, float beta, const uint64_t* seeds, void* stream)
{
    return set_compress(set, seeds, 1.0f - beta, beta, stream);
}

flora_status flora_set_decompress_apply(flora_set* set, const uint64_t* seeds, float lr, float scale, void* stream)
{
    if (!set || !seeds) return FLORA_ERR_NULL;
    if (!set->has_W) return FLORA_ERR_UNSUPPORTED;
    if (set->tc.decompress_ready && g_force_path.load() != 1)
        return tc_set_decompress(set->tc, seeds, lr * scale, as_stream(stream), g_launches);
    for (size_t i = 0; i < set->W.size(); ++i) {
        if (set->W[i].rows == 0 || set->W[i].cols == 0) continue;
        flora_status st = simt_decompress(&set->W[i], &set->S[i], seeds[i], lr * scale, as_stream(stream));
        if (st) return st;
    }
    return FLORA_OK;
}

// dst.S[i] <- b dst.S[i] + a src[i] (A(old_i) A(new_i)^T) for every matrix of the set `dst`.
static flora_status set_transfer(flora_set* set, const std::vector<flora_mat>& src, const TcMatrix* src_mats, const uint64_t* seeds_old,
                                 const uint64_t* seeds_new, float a, float b, void* stream, void** release_later = nullptr)
{
    if (release_later) *release_later = nullptr;
    if (!set || !seeds_old || !seeds_new) return FLORA_ERR_NULL;
    const std::vector<flora_mat>& big = set->has_G ? set->G : set->W;
    const int r = set->r;
    float* T = nullptr;
    if (set->S.empty()) return FLORA_OK;
    bool all_bf16 = g_force_path.load() != 1;
    for (const auto& g : big) all_bf16 = all_bf16 && g.dtype == FLORA_BF16 && g.cols <= 0x7FFFFFFF && g.rows <= 0x7FFFFFFF;
    if (all_bf16) {
        // one gram launch and one apply launch over the whole set
        std::vector<GramJob> jobs;
        for (size_t i = 0; i < set->S.size(); ++i) {
            if (set->S[i].rows == 0) continue;
            jobs.push_back(GramJob{nullptr, (float*)set->S[i].data, (const float*)src[i].data, set->S[i].ld, src[i].ld,
                                   (int32_t)set->S[i].rows, (int32_t)big[i].cols, seeds_old[i], seeds_new[i], (int32_t)i, 0});
        }
        return transfer_tc(jobs, r, a, b, as_stream(stream), g_launches, set->tc.d_mats, src_mats, nullptr, release_later);
    }
    if (scratch_alloc((void**)&T, sizeof(float) * r * r, as_stream(stream)) != cudaSuccess) {
        cudaGetLastError();
        return FLORA_ERR_ALLOC;
    }
    flora_status st = FLORA_OK;
    for (size_t i = 0; i < set->S.size() && st == FLORA_OK; ++i) {
        if (set->S[i].rows == 0) continue;
        st = transfer_with_scratch(&set->S[i], &src[i], big[i].cols, big[i].dtype, seeds_old[i], seeds_new[i], a, b, T, as_stream(stream));
    }
    if (cudaFreeAsync(T, as_stream(stream)) != cudaSuccess && st == FLORA_OK) st = FLORA_ERR_CUDA;
    return st;
}

flora_status flora_set_resample_transfer(flora_set* set, const uint64_t* seeds_old, const uint64_t* seeds_new, void* stream)
{
    if (!set) return FLORA_ERR_NULL;
    return set_transfer(set, set->S, set->tc.d_mats, seeds_old, seeds_new, 1.0f, 0.0f, stream);
}

flora_status flora_set_transfer_axpby(flora_set* dst, const flora_set* src, const uint64_t* seeds_old, const uint64_t* seeds_new, float a, float b,
                                      void* stream)
{
    if (!dst || !src) return FLORA_ERR_NULL;
    if (src->S.size() != dst->S.size() || src->r != dst->r) return FLORA_ERR_SHAPE;
    for (size_t i = 0; i < dst->S.size(); ++i)
        if (src->S[i].rows != dst->S[i].rows) return FLORA_ERR_SHAPE;
    return set_transfer(dst, src->S, src->tc.d_mats, seeds_old, seeds_new, a, b, stream);
}

flora_status flora_set_momentum_step_resampled(flora_set* set, float beta, const uint64_t* seeds_old, const uint64_t* seeds_new, void* stream)
{
    if (!set || !seeds_old || !seeds_new) return FLORA_ERR_NULL;
    if (!set->has_G) return FLORA_ERR_UNSUPPORTED;
    // the compression goes right behind the transfer's last kernel and starts while that one still runs (it waits itself
    // before it touches a sketch); the transfer's scratch is handed back after it has been launched
    void* scratch = nullptr;
    flora_status st = set_transfer(set, set->S, set->tc.d_mats, seeds_old, seeds_new, beta, 0.0f, stream, &scratch);
    if (st == FLORA_OK) st = set_compress(set, seeds_new, 1.0f - beta, 1.0f, stream, scratch != nullptr);
    if (scratch && cudaFreeAsync(scratch, as_stream(stream)) != cudaSuccess && st == FLORA_OK) st = FLORA_ERR_CUDA;
    return st;
}

flora_status flora_set_zero_state(flora_set* set, void* stream)
{
    if (!set) return FLORA_ERR_NULL;
    if (set->tc.d_mats && g_force_path.load() != 1) return tc_set_zero(set->tc, as_stream(stream), g_launches);
    for (auto& s : set->S) {
        if (s.rows == 0) continue;
        cudaError_t e = cudaMemset2DAsync(s.data, sizeof(float) * s.ld, 0, sizeof(float) * s.cols, (size_t)s.rows, as_stream(stream));
        if (e != cudaSuccess) return FLORA_ERR_CUDA;
    }
    return FLORA_OK;
}

flora_status flora_set_upload_gradients(flora_set* set, const void* const* host_G, void* stream)
{
    if (!set || !host_G) return FLORA_ERR_NULL;
    if (!set->has_G) return FLORA_ERR_UNSUPPORTED;
    for (size_t i = 0; i < set->G.size(); ++i) {
        const flora_mat& g = set->G[i];
        if (g.rows == 0 || g.cols == 0) continue;
        if (!host_G[i]) return FLORA_ERR_NULL;
        const size_t es = elem_size(g.dtype);
        // a densely stored matrix is one plain copy; a strided one goes row by row
        cudaError_t e = g.ld == g.cols
                            ? cudaMemcpyAsync(g.data, host_G[i], es * (size_t)g.rows * (size_t)g.cols, cudaMemcpyHostToDevice, as_stream(stream))
                            : cudaMemcpy2DAsync(g.data, es * g.ld, host_G[i], es * g.cols, es * g.cols, (size_t)g.rows, cudaMemcpyHostToDevice,
                                                as_stream(stream));
        if (e != cudaSuccess) return FLORA_ERR_CUDA;
    }
    return FLORA_OK;
}

flora_status flora_set_compress_accumulate_from_host(flora_set* set, const void* const* host_G, const uint64_t* seeds, void* stream)
{
    if (!seeds) return FLORA_ERR_NULL;
    flora_status st = flora_set_upload_gradients(set, host_G, stream);
    if (st) return st;
    return flora_set_compress_accumulate(set, seeds, stream);
}

flora_status flora_set_read_weights_to_host(flora_set* set, void* const* host_W, void* stream)
{
    if (!set || !host_W) return FLORA_ERR_NULL;
    if (!set->has_W) return FLORA_ERR_UNSUPPORTED;
    for (size_t i = 0; i < set->W.size(); ++i) {
        const flora_mat& w = set->W[i];
        if (w.rows == 0 || w.cols == 0) continue;
        if (!host_W[i]) return FLORA_ERR_NULL;
        const size_t es = elem_size(w.dtype);
        cudaError_t e = w.ld == w.cols
                            ? cudaMemcpyAsync(host_W[i], w.data, es * (size_t)w.rows * (size_t)w.cols, cudaMemcpyDeviceToHost, as_stream(stream))
                            : cudaMemcpy2DAsync(host_W[i], es * w.cols, w.data, es * w.ld, es * w.cols, (size_t)w.rows, cudaMemcpyDeviceToHost,
                                                as_stream(stream));
        if (e != cudaSuccess) return FLORA_ERR_CUDA;
    }
    return FLORA_OK;
}

// ------------------------------------------------------------------------------------------------
// host sequencing
// ------------------------------------------------------------------------------------------------
uint64_t flora_derive_seed(uint64_t base, uint64_t matrix, uint64_t epoch)
{
    uint64_t z = base ^ (matrix * 0x9E3779B97F4A7C15ull) ^ (epoch * 0xD1B54A32D192ED03ull);
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

int flora_resamples_at(int64_t t, int64_t kappa) { return (kappa > 0 && t >= 0 && t % kappa == 0) ? 1 : 0; }

// ------------------------------------------------------------------------------------------------
// diagnostics
// ------------------------------------------------------------------------------------------------
void flora_debug_force_path(int path) { g_force_path.store(path == 1 ? 1 : 0); }

void flora_set_deterministic(int on) { deterministic_flag().store(on ? 1 : 0); }

flora_status flora_debug_plan(const int64_t* rows, const int64_t* cols, int64_t count, int32_t r, int32_t which, int32_t* items, int64_t capacity,
                              int64_t* n_items, int32_t* params)
{
    if (!rows || !cols || !n_items || !params || (capacity > 0 && !items)) return FLORA_ERR_NULL;
    if (count < 0 || capacity < 0) return FLORA_ERR_SHAPE;
    if (r < 1 || r > 256) return FLORA_ERR_RANK;
    std::vector<flora_mat> mats((size_t)count);
    for (int64_t i = 0; i < count; ++i) {
        if (rows[i] < 0 || cols[i] < 0 || rows[i] > 0x7FFFFF00ll || cols[i] > 0x7FFFFF00ll) return FLORA_ERR_SHAPE;
        mats[(size_t)i] = flora_mat{nullptr, rows[i], cols[i], cols[i], FLORA_BF16};
    }
    TcSet set;
    set.count = (int)count;
    set.r = r;
    const int width = which == 0 ? 6 : which == 2 ? 1 : 4;
    if (which == 2) {
        // the slot table of the persistent compression kernel (ranks above 64): per launch, one first-unit index per
        // slot and the unit count; empty for the ranks that run one CTA per item
        plan_compress(set, mats, r);
        *n_items = (int64_t)set.h_slots.size();
        const int32_t p[8] = {set.T, set.S, set.gstages, set.astages, set.GW, set.P, (int32_t)(set.k1_launch_begin.size() - 1), (int32_t)set.k1_smem};
        memcpy(params, p, sizeof(p));
        for (int64_t i = 0; i < std::min<int64_t>(*n_items, capacity); ++i) items[i] = set.h_slots[(size_t)i];
    } else if (which == 0) {
        plan_compress(set, mats, r);
        *n_items = (int64_t)set.h_k1.size();
        const int32_t p[8] = {set.T, set.S, set.gstages, set.astages, set.GW, set.P, (int32_t)(set.k1_launch_begin.size() - 1), (int32_t)set.k1_smem};
        memcpy(params, p, sizeof(p));
        for (int64_t i = 0; i < std::min<int64_t>(*n_items, capacity); ++i) {
            const K1Item& it = set.h_k1[(size_t)i];
            const int32_t v[6] = {it.mat, it.row0, it.tiles, it.kstep0, it.ksteps, it.direct};
            memcpy(items + i * width, v, sizeof(v));
        }
    } else {
        plan_decompress(set, mats, r);
        *n_items = (int64_t)set.h_k2.size();
        const int32_t p[8] = {set.bn, set.slots, set.cstages, set.k2_nslabs, set.k2_gw, set.k2_bf16 ? 1 : 0, (int32_t)(set.k2_launch_begin.size() - 1),
                              (int32_t)set.k2_smem};
        memcpy(params, p, sizeof(p));
        for (int64_t i = 0; i < std::min<int64_t>(*n_items, capacity); ++i) {
            const K2Item& it = set.h_k2[(size_t)i];
            const int32_t v[4] = {it.mat, it.col0, it.row0, it.tiles};
            memcpy(items + i * width, v, sizeof(v));
        }
    }
    cudaGetLastError();        // without a device the occupancy queries inside the planners fail and fall back; leave no sticky error
    return FLORA_OK;
}
uint64_t flora_launch_count(void) { return g_launches.load(); }

flora_status flora_device_status(void)
{
    int word = 0;
    if (!tc_read_and_clear_error(&word)) return FLORA_ERR_CUDA;
    return word ? FLORA_ERR_TIMEOUT : FLORA_OK;
}

flora_status flora_debug_wait_timeout_selftest(void* stream)
{
    int* flag = nullptr;
    if (scratch_alloc((void**)&flag, sizeof(int), as_stream(stream)) != cudaSuccess) {
        cudaGetLastError();
        return FLORA_ERR_ALLOC;
    }
    cudaMemsetAsync(flag, 0, sizeof(int), as_stream(stream));
    wait_timeout_selftest_kernel<<<1, 32, 0, as_stream(stream)>>>(flag);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    int gave_up = 0;
    cudaError_t e = cudaMemcpyAsync(&gave_up, flag, sizeof(int), cudaMemcpyDeviceToHost, as_stream(stream));
    if (e == cudaSuccess) e = cudaStreamSynchronize(as_stream(stream));
    cudaFreeAsync(flag, as_stream(stream));
    if (e != cudaSuccess) return FLORA_ERR_CUDA;
    return gave_up ? FLORA_ERR_TIMEOUT : FLORA_OK;
}

const char* flora_status_string(flora_status s)
{
    switch (s) {
        case FLORA_OK: return "ok";
        case FLORA_ERR_NULL: return "null pointer";
        case FLORA_ERR_SHAPE: return "bad shape or leading dimension";
        case FLORA_ERR_DTYPE: return "dtype not allowed here";
        case FLORA_ERR_ALIGN: return "misaligned pointer";
        case FLORA_ERR_RANK: return "rank out of range or inconsistent";
        case FLORA_ERR_CUDA: return "CUDA call failed";
        case FLORA_ERR_TIMEOUT: return "device-side wait timed out";
        case FLORA_ERR_UNSUPPORTED: return "unsupported arguments";
        case FLORA_ERR_ALLOC: return "allocation failed";
    }
    return "unknown status";
}

int flora_version(void) { return 100; }

}  // extern "C"
