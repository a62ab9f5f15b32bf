// C ABI of the library: argument validation and kernel launches (see include/dq.h).
#include <atomic>
#include <cstdio>
#include <cstring>
#include <new>

#include "dq_internal.h"

namespace {

thread_local char g_cuda_error[256] = "";

int cuda_fail(cudaError_t e, const char* where) {
    std::snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", where, cudaGetErrorString(e));
    return DQ_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Process-wide options (dq_set_option); a negative value means "library default".
std::atomic<long long> g_opt_step_poll_limit{-1};
std::atomic<long long> g_opt_encode_batch_min{-1};

// Checks every attention entry point makes on the tables and the arrays they describe: values carry
// no window mean, both tables group heads the same way and Hkv is a whole number of groups (the
// kernels derive the container layout from them), the mean arrays cover every addressable
// position, and the alignments the 16-byte copies need.
int check_attn_tables(const dq_tables* tk, const dq_tables* tv, int Hkv, const uint8_t* k_cont, const uint8_t* v_cont,
                      const int8_t* k_mean_q, const float* k_mean_scale, int max_windows, int max_pages,
                      const void* out_bf16, const float* out_f32) {
    if (!tk || !tv || !k_cont || !v_cont) return DQ_ERR_ARG;
    if (tv->info.has_mean) return DQ_ERR_UNSUPPORTED;
    if (tk->info.heads_per_stream != tv->info.heads_per_stream) return DQ_ERR_UNSUPPORTED;
    if (tk->info.sigma_bits != tv->info.sigma_bits) return DQ_ERR_UNSUPPORTED;   // one state width per cache
    if (tk->info.pair_symbols != tv->info.pair_symbols) return DQ_ERR_UNSUPPORTED;   // one symbol alphabet kind per cache
    if (Hkv <= 0 || Hkv % tk->info.heads_per_stream != 0) return DQ_ERR_ARG;
    if (tk->info.has_mean && (!k_mean_q || !k_mean_scale || max_windows <= 0)) return DQ_ERR_ARG;
    if (tk->info.has_mean && (long long)max_windows * DQ_WINDOW_TOKENS < (long long)max_pages * DQ_PAGE_TOKENS)
        return DQ_ERR_ARG;  // every addressable position needs a window slot
    if (!aligned16(k_cont) || !aligned16(v_cont) || (tk->info.has_mean && !aligned16(k_mean_q))) return DQ_ERR_ARG;
    if ((out_bf16 && (reinterpret_cast<uintptr_t>(out_bf16) & 7u)) || (out_f32 && !aligned16(out_f32)))
        return DQ_ERR_ARG;
    return DQ_OK;
}

}  // namespace

int dq_opt_step_poll_limit(int dflt) {
    const long long v = g_opt_step_poll_limit.load(std::memory_order_relaxed);
    return v < 0 ? dflt : (int)v;
}
long long dq_opt_encode_batch_min(long long dflt) {
    const long long v = g_opt_encode_batch_min.load(std::memory_order_relaxed);
    return v < 0 ? dflt : v;
}

extern "C" {

int dq_build_tables(int levels, double bits_per_elem, const dq_table_opts* opts, dq_tables** out) {
    if (!opts || !out) return DQ_ERR_ARG;
    dq_tables* t = new (std::nothrow) dq_tables;
    if (!t) return DQ_ERR_ARG;
    const int rc = dq_host_build(levels, bits_per_elem, opts, t);
    if (rc != DQ_OK) {
        delete t;
        return rc;
    }
    *out = t;
    return DQ_OK;
}

void dq_free_tables(dq_tables* t) { delete t; }

int dq_tables_info(const dq_tables* t, dq_table_info* out) {
    if (!t || !out) return DQ_ERR_ARG;
    *out = t->info;
    return DQ_OK;
}

int dq_encode_tokens_rope(const dq_tables* tk, const dq_tables* tv, const void* k_bf16, const void* v_bf16,
                          int T, int Hkv, const int32_t* seq_id, const int32_t* pos, const int32_t* slot,
                          uint8_t* k_cont, uint8_t* v_cont, int8_t* k_mean_q, float* k_mean_scale,
                          int max_windows, int mean_mode, const float* rope_cos, const float* rope_sin,
                          int rope_style, uint32_t* status, void* cuda_stream) {
    if (T < 0 || Hkv <= 0 || (!tk && !tv)) return DQ_ERR_ARG;
    if (rope_style != 0 && rope_style != DQ_ROPE_HALF && rope_style != DQ_ROPE_PAIRS) return DQ_ERR_ARG;
    if (rope_style != 0 && (!rope_cos || !rope_sin || !aligned16(rope_cos) || !aligned16(rope_sin))) return DQ_ERR_ARG;
    if (!seq_id || !pos || !slot) return DQ_ERR_ARG;
    if (tk && (!k_bf16 || !k_cont)) return DQ_ERR_ARG;
    if (tv && (!v_bf16 || !v_cont)) return DQ_ERR_ARG;
    if (mean_mode != DQ_MEAN_COMPUTE && mean_mode != DQ_MEAN_REUSE) return DQ_ERR_ARG;
    const bool k_mean = tk && tk->info.has_mean;
    if (k_mean && (!k_mean_q || !k_mean_scale || max_windows <= 0)) return DQ_ERR_ARG;
    if (tv && tv->info.has_mean) return DQ_ERR_UNSUPPORTED;  // only keys carry window means
    {
        const int hs = tk ? tk->info.heads_per_stream : tv->info.heads_per_stream;
        if (tk && tv && tk->info.heads_per_stream != tv->info.heads_per_stream) return DQ_ERR_UNSUPPORTED;
        if (tk && tv && tk->info.pair_symbols != tv->info.pair_symbols) return DQ_ERR_UNSUPPORTED;
        if (Hkv % hs != 0) return DQ_ERR_ARG;
    }
    if ((k_bf16 && (reinterpret_cast<uintptr_t>(k_bf16) & 7u)) ||
        (v_bf16 && (reinterpret_cast<uintptr_t>(v_bf16) & 7u)) ||
        (k_mean && (reinterpret_cast<uintptr_t>(k_mean_q) & 3u)))
        return DQ_ERR_ARG;
    if (T == 0) return DQ_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e;
    if (k_mean && mean_mode == DQ_MEAN_COMPUTE) {
        e = dq_launch_means(tk->dev, k_bf16, T, Hkv, seq_id, pos, k_mean_q, k_mean_scale, max_windows,
                            mean_mode, rope_cos, rope_sin, rope_style, st);
        if (e != cudaSuccess) return cuda_fail(e, "window means");
    }
    // keys and values go through one launch; in DQ_MEAN_REUSE mode the encoder warp of a
    // window's first token carries the previous mean forward itself
    DqEncodeArgs a;
    a.k_bf16 = k_bf16; a.v_bf16 = v_bf16; a.seq_id = seq_id; a.pos = pos; a.slot = slot;
    a.k_cont = k_cont; a.v_cont = v_cont; a.mean_q = k_mean_q; a.mean_scale = k_mean_scale;
    a.status = status; a.T = T; a.Hkv = Hkv; a.max_windows = max_windows; a.mean_mode = mean_mode;
    a.do_k = tk ? 1 : 0; a.do_v = tv ? 1 : 0;
    a.rope_cos = rope_cos; a.rope_sin = rope_sin; a.rope_style = rope_style;
    a.step_seq_lens = nullptr; a.step_flags = nullptr;
    e = dq_launch_encode(tk ? tk->dev : tv->dev, tv ? tv->dev : tk->dev, tk ? tk->penc : tv->penc, tv ? tv->penc : tk->penc, a, st);
    if (e != cudaSuccess) return cuda_fail(e, "encode");
    return DQ_OK;
}

int dq_encode_tokens(const dq_tables* tk, const dq_tables* tv, const void* k_bf16, const void* v_bf16,
                     int T, int Hkv, const int32_t* seq_id, const int32_t* pos, const int32_t* slot,
                     uint8_t* k_cont, uint8_t* v_cont, int8_t* k_mean_q, float* k_mean_scale,
                     int max_windows, int mean_mode, uint32_t* status, void* cuda_stream) {
    return dq_encode_tokens_rope(tk, tv, k_bf16, v_bf16, T, Hkv, seq_id, pos, slot, k_cont, v_cont, k_mean_q,
                                 k_mean_scale, max_windows, mean_mode, nullptr, nullptr, 0, status, cuda_stream);
}

size_t dq_decode_workspace_bytes(int B, int Hq, int max_pages) {
    if (B <= 0 || Hq <= 0 || max_pages <= 0) return 0;
    return dq_attn_workspace_bytes(B, Hq, max_pages);
}

static int check_attn_common(const void* q, const int32_t* page_table, int max_pages,
                             const int32_t* seq_lens, int B, int Hq, int Hkv, const void* out_a,
                             const void* out_b, void* workspace, size_t workspace_bytes) {
    if (!q || !page_table || !seq_lens || (!out_a && !out_b) || !workspace) return DQ_ERR_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || max_pages <= 0) return DQ_ERR_ARG;
    if (Hq % Hkv != 0) return DQ_ERR_ARG;
    if (Hq / Hkv > DQ_MAX_GROUP || B > 4096) return DQ_ERR_UNSUPPORTED;
    if (!aligned16(workspace) || (reinterpret_cast<uintptr_t>(q) & 7u)) return DQ_ERR_ARG;
    if (workspace_bytes < dq_attn_workspace_bytes(B, Hq, max_pages)) return DQ_ERR_WORKSPACE;
    return DQ_OK;
}

int dq_decode_attention_multi(const dq_tables* tk, const dq_tables* tv, const void* q_bf16, int q_len,
                              const uint8_t* k_cont, const uint8_t* v_cont, const int8_t* k_mean_q,
                              const float* k_mean_scale, int max_windows, const int32_t* page_table,
                              int max_pages, const int32_t* seq_lens, const void* resid_k_bf16,
                              const void* resid_v_bf16, const int32_t* resid_lens, int resid_cap, int B, int Hq,
                              int Hkv, float sm_scale, void* out_bf16, float* out_f32, void* workspace,
                              size_t workspace_bytes, void* cuda_stream) {
    if (!tk || !tv || !k_cont || !v_cont) return DQ_ERR_ARG;
    if (q_len < 1) return DQ_ERR_ARG;
    if (resid_k_bf16 || resid_v_bf16 || resid_lens) {
        if (!resid_k_bf16 || !resid_v_bf16 || !resid_lens || resid_cap <= 0) return DQ_ERR_ARG;
        if ((reinterpret_cast<uintptr_t>(resid_k_bf16) & 7u) || (reinterpret_cast<uintptr_t>(resid_v_bf16) & 7u))
            return DQ_ERR_ARG;
    }
    int rc = check_attn_common(q_bf16, page_table, max_pages, seq_lens, B, Hq, Hkv, out_bf16, out_f32,
                               workspace, workspace_bytes);
    if (rc != DQ_OK) return rc;
    {   // one pass holds DQ_MAX_GROUP rows per KV head; more query tokens take more passes over the same scratch
        const int per_pass = DQ_MAX_GROUP / (Hq / Hkv);
        const int pass_tokens = q_len < per_pass ? q_len : per_pass;
        if (workspace_bytes < dq_attn_workspace_bytes(B, Hq * pass_tokens, max_pages)) return DQ_ERR_WORKSPACE;
    }
    rc = check_attn_tables(tk, tv, Hkv, k_cont, v_cont, k_mean_q, k_mean_scale, max_windows, max_pages, out_bf16, out_f32);
    if (rc != DQ_OK) return rc;
    DqAttnArgs a;
    a.q_bf16 = q_bf16; a.k_cont = k_cont; a.v_cont = v_cont;
    a.mean_q = k_mean_q; a.mean_scale = k_mean_scale;
    a.page_table = page_table; a.seq_lens = seq_lens;
    a.out_bf16 = out_bf16; a.out_f32 = out_f32; a.workspace = workspace;
    a.max_windows = max_windows; a.max_pages = max_pages;
    a.B = B; a.Hq = Hq; a.Hkv = Hkv; a.sm_scale = sm_scale;
    a.resid_k = resid_k_bf16; a.resid_v = resid_v_bf16; a.resid_lens = resid_lens; a.resid_cap = resid_cap;
    a.q_len = q_len;
    a.fused = 0;
    const cudaError_t e = dq_launch_attention(tk->dev, tv->dev, a, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(e, "decode attention");
    return DQ_OK;
}

int dq_decode_attention_residual(const dq_tables* tk, const dq_tables* tv, const void* q_bf16,
                                 const uint8_t* k_cont, const uint8_t* v_cont, const int8_t* k_mean_q,
                                 const float* k_mean_scale, int max_windows, const int32_t* page_table,
                                 int max_pages, const int32_t* seq_lens, const void* resid_k_bf16,
                                 const void* resid_v_bf16, const int32_t* resid_lens, int resid_cap, int B, int Hq,
                                 int Hkv, float sm_scale, void* out_bf16, float* out_f32, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream) {
    return dq_decode_attention_multi(tk, tv, q_bf16, 1, k_cont, v_cont, k_mean_q, k_mean_scale, max_windows, page_table,
                                     max_pages, seq_lens, resid_k_bf16, resid_v_bf16, resid_lens, resid_cap, B, Hq, Hkv,
                                     sm_scale, out_bf16, out_f32, workspace, workspace_bytes, cuda_stream);
}

int dq_decode_attention(const dq_tables* tk, const dq_tables* tv, const void* q_bf16,
                        const uint8_t* k_cont, const uint8_t* v_cont, const int8_t* k_mean_q,
                        const float* k_mean_scale, int max_windows, const int32_t* page_table,
                        int max_pages, const int32_t* seq_lens, int B, int Hq, int Hkv, float sm_scale,
                        void* out_bf16, float* out_f32, void* workspace, size_t workspace_bytes,
                        void* cuda_stream) {
    return dq_decode_attention_residual(tk, tv, q_bf16, k_cont, v_cont, k_mean_q, k_mean_scale, max_windows,
                                        page_table, max_pages, seq_lens, nullptr, nullptr, nullptr, 0, B, Hq, Hkv,
                                        sm_scale, out_bf16, out_f32, workspace, workspace_bytes, cuda_stream);
}

int dq_decode_attention_static(const dq_tables* tk, const dq_tables* tv, const void* q_bf16,
                               const uint8_t* k_cont, const uint8_t* v_cont, const int8_t* k_mean_q,
                               const float* k_mean_scale, int max_windows, const int32_t* page_table,
                               int max_pages, const int32_t* seq_lens, int B, int Hq, int Hkv, float sm_scale,
                               void* out_bf16, float* out_f32, void* cuda_stream) {
    if (!tk || !tv || !k_cont || !v_cont) return DQ_ERR_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || max_pages <= 0) return DQ_ERR_ARG;
    int rc = check_attn_tables(tk, tv, Hkv, k_cont, v_cont, k_mean_q, k_mean_scale, max_windows, max_pages, out_bf16, out_f32);
    if (rc != DQ_OK) return rc;   // decided on the host, before any CUDA call
    const size_t need = dq_attn_workspace_bytes(B, Hq, max_pages);
    if (need > (size_t)DQ_STATIC_SCRATCH_BYTES) {  // decided on the host, before any CUDA call
        std::snprintf(g_cuda_error, sizeof g_cuda_error,
                      "dq_decode_attention_static: the built-in scratch holds %zu bytes, this call needs %zu "
                      "(B=%d, Hq=%d, max_pages=%d); use dq_decode_attention with a workspace",
                      (size_t)DQ_STATIC_SCRATCH_BYTES, need, B, Hq, max_pages);
        return DQ_ERR_WORKSPACE;
    }
    void* scratch = nullptr;
    cudaError_t e = dq_attn_static_scratch(&scratch);
    if (e != cudaSuccess) return cuda_fail(e, "static scratch address");
    rc = check_attn_common(q_bf16, page_table, max_pages, seq_lens, B, Hq, Hkv, out_bf16, out_f32, scratch,
                           (size_t)DQ_STATIC_SCRATCH_BYTES);
    if (rc != DQ_OK) return rc;
    DqAttnArgs a;
    a.q_bf16 = q_bf16; a.k_cont = k_cont; a.v_cont = v_cont;
    a.mean_q = k_mean_q; a.mean_scale = k_mean_scale;
    a.page_table = page_table; a.seq_lens = seq_lens;
    a.out_bf16 = out_bf16; a.out_f32 = out_f32; a.workspace = scratch;
    a.max_windows = max_windows; a.max_pages = max_pages;
    a.B = B; a.Hq = Hq; a.Hkv = Hkv; a.sm_scale = sm_scale;
    a.resid_k = nullptr; a.resid_v = nullptr; a.resid_lens = nullptr; a.resid_cap = 0;
    a.q_len = 1;
    a.fused = 0;
    e = dq_launch_attention_static(tk->dev, tv->dev, a, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(e, "decode attention (static scratch)");
    return DQ_OK;
}

int dq_decode_tokens(const dq_tables* t, const uint8_t* cont, const int8_t* mean_q, const float* mean_scale,
                     int max_windows, const int32_t* seq_id, const int32_t* pos, const int32_t* slot, int T,
                     int Hkv, uint8_t* symbols, float* dequant, void* cuda_stream) {
    if (!t || !cont || !slot || T < 0 || Hkv <= 0 || (!symbols && !dequant)) return DQ_ERR_ARG;
    if (t->info.has_mean && mean_q && (!mean_scale || !seq_id || !pos || max_windows <= 0)) return DQ_ERR_ARG;
    if (Hkv % t->info.heads_per_stream != 0) return DQ_ERR_ARG;   // the container layout has Hkv / hs groups
    if (T == 0) return DQ_OK;
    const cudaError_t e = dq_launch_decode_tokens(t->dev, cont, mean_q, mean_scale, max_windows, seq_id, pos,
                                                  slot, T, Hkv, symbols, dequant,
                                                  static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(e, "decode tokens");
    return DQ_OK;
}

int dq_bf16_decode_attention(const void* q_bf16, const void* k_bf16_pages, const void* v_bf16_pages,
                             const int32_t* page_table, int max_pages, const int32_t* seq_lens, int B,
                             int Hq, int Hkv, float sm_scale, void* out_bf16, void* workspace,
                             size_t workspace_bytes, void* cuda_stream) {
    if (!k_bf16_pages || !v_bf16_pages) return DQ_ERR_ARG;
    int rc = check_attn_common(q_bf16, page_table, max_pages, seq_lens, B, Hq, Hkv, out_bf16, nullptr,
                               workspace, workspace_bytes);
    if (rc != DQ_OK) return rc;
    if (!aligned16(k_bf16_pages) || !aligned16(v_bf16_pages) || (reinterpret_cast<uintptr_t>(out_bf16) & 7u))
        return DQ_ERR_ARG;
    DqAttnArgs a;
    std::memset(&a, 0, sizeof a);
    a.q_bf16 = q_bf16; a.page_table = page_table; a.seq_lens = seq_lens;
    a.out_bf16 = out_bf16; a.workspace = workspace;
    a.max_pages = max_pages; a.B = B; a.Hq = Hq; a.Hkv = Hkv; a.sm_scale = sm_scale;
    const cudaError_t e = dq_launch_bf16_attention(a, k_bf16_pages, v_bf16_pages,
                                                   static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(e, "bf16 decode attention");
    return DQ_OK;
}

int dq_decode_step(const dq_tables* tk, const dq_tables* tv, const void* k_new_bf16, const void* v_new_bf16,
                   const int32_t* slot_new, const void* q_bf16, uint8_t* k_cont, uint8_t* v_cont, int8_t* k_mean_q,
                   float* k_mean_scale, int max_windows, const int32_t* page_table, int max_pages,
                   const int32_t* seq_lens, int B, int Hq, int Hkv, float sm_scale, void* out_bf16, float* out_f32,
                   void* workspace, size_t workspace_bytes, uint32_t* status, void* cuda_stream) {
    if (!tk || !tv || !k_new_bf16 || !v_new_bf16 || !slot_new || !k_cont || !v_cont) return DQ_ERR_ARG;
    int rc = check_attn_common(q_bf16, page_table, max_pages, seq_lens, B, Hq, Hkv, out_bf16, out_f32, workspace,
                               workspace_bytes);
    if (rc != DQ_OK) return rc;
    if (tk->info.heads_per_stream != 1 || tv->info.heads_per_stream != 1) return DQ_ERR_UNSUPPORTED;
    rc = check_attn_tables(tk, tv, Hkv, k_cont, v_cont, k_mean_q, k_mean_scale, max_windows, max_pages, out_bf16, out_f32);
    if (rc != DQ_OK) return rc;
    if ((reinterpret_cast<uintptr_t>(k_new_bf16) & 7u) || (reinterpret_cast<uintptr_t>(v_new_bf16) & 7u)) return DQ_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    DqEncodeArgs e;
    std::memset(&e, 0, sizeof e);
    e.k_bf16 = k_new_bf16; e.v_bf16 = v_new_bf16; e.slot = slot_new;
    e.k_cont = k_cont; e.v_cont = v_cont; e.mean_q = k_mean_q; e.mean_scale = k_mean_scale;
    e.status = status; e.T = B; e.Hkv = Hkv; e.max_windows = max_windows; e.mean_mode = DQ_MEAN_REUSE;
    e.do_k = 1; e.do_v = 1;
    e.step_seq_lens = seq_lens; e.step_flags = dq_attn_workspace_flags(workspace);
    cudaError_t ce = dq_launch_encode(tk->dev, tv->dev, tk->penc, tv->penc, e, st);
    if (ce != cudaSuccess) return cuda_fail(ce, "decode step: encode");
    DqAttnArgs a;
    std::memset(&a, 0, sizeof a);
    a.q_bf16 = q_bf16; a.k_cont = k_cont; a.v_cont = v_cont;
    a.mean_q = k_mean_q; a.mean_scale = k_mean_scale;
    a.page_table = page_table; a.seq_lens = seq_lens;
    a.out_bf16 = out_bf16; a.out_f32 = out_f32; a.workspace = workspace;
    a.max_windows = max_windows; a.max_pages = max_pages;
    a.B = B; a.Hq = Hq; a.Hkv = Hkv; a.sm_scale = sm_scale;
    ce = dq_launch_step(tk->dev, tv->dev, e, a, st);
    if (ce != cudaSuccess) return cuda_fail(ce, "decode step: attention");
    return DQ_OK;
}

int dq_window_append(const void* k_bf16, const void* v_bf16, void* resid_k_bf16, void* resid_v_bf16,
                     int32_t* resid_lens, int resid_cap, int B, int Hkv, void* cuda_stream) {
    if (!k_bf16 || !v_bf16 || !resid_k_bf16 || !resid_v_bf16 || !resid_lens) return DQ_ERR_ARG;
    if (B < 0 || Hkv <= 0 || resid_cap <= 0) return DQ_ERR_ARG;
    if (!aligned16(k_bf16) || !aligned16(v_bf16) || !aligned16(resid_k_bf16) || !aligned16(resid_v_bf16)) return DQ_ERR_ARG;
    const cudaError_t e = dq_launch_window_append(k_bf16, v_bf16, resid_k_bf16, resid_v_bf16, resid_lens, resid_cap, B, Hkv,
                                                  static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(e, "window append");
    return DQ_OK;
}

int dq_set_option(int key, long long value) {
    if (value < 0) value = -1;
    switch (key) {
        case DQ_OPT_STEP_POLL_LIMIT:
            if (value > (1LL << 24)) return DQ_ERR_ARG;
            g_opt_step_poll_limit.store(value, std::memory_order_relaxed);
            return DQ_OK;
        case DQ_OPT_ENCODE_BATCH_MIN:
            g_opt_encode_batch_min.store(value, std::memory_order_relaxed);
            return DQ_OK;
        default: return DQ_ERR_ARG;
    }
}

long long dq_get_option(int key) {
    switch (key) {
        case DQ_OPT_STEP_POLL_LIMIT: return g_opt_step_poll_limit.load(std::memory_order_relaxed);
        case DQ_OPT_ENCODE_BATCH_MIN: return g_opt_encode_batch_min.load(std::memory_order_relaxed);
        default: return -1;
    }
}

int dq_microbench_decode_loop(const dq_tables* t, const uint8_t* bytes, size_t nbytes, int ctas, int threads, int chains,
                              int reps, uint32_t* out, void* cuda_stream) {
    if (!t || !bytes || !out || nbytes < 4096 || nbytes > 0xffffffffull) return DQ_ERR_ARG;
    if (ctas <= 0 || reps <= 0 || (chains != 1 && chains != 2)) return DQ_ERR_ARG;
    if (threads < 32 || threads > 1024 || threads % 32 != 0) return DQ_ERR_ARG;
    const cudaError_t e = dq_launch_microbench_decode_loop(t->dev, bytes, nbytes, ctas, threads, chains, reps, out,
                                                           static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(e, "decode-loop microbenchmark");
    return DQ_OK;
}

void dq_profile_enable(int on) { dq_attn_profile_enable(on); }

int dq_profile_read(float* ms_out, int max_records) {
    if (!ms_out || max_records <= 0) return 0;
    return dq_attn_profile_read(ms_out, max_records);
}

const char* dq_strerror(int code) {
    switch (code) {
        case DQ_OK: return "ok";
        case DQ_ERR_ARG: return "invalid argument";
        case DQ_ERR_INFEASIBLE: return "levels do not fit the container budget";
        case DQ_ERR_UNSUPPORTED: return "unsupported configuration";
        case DQ_ERR_WORKSPACE: return "workspace too small";
        case DQ_ERR_CUDA: return "CUDA error";
        default: return "unknown error";
    }
}

const char* dq_last_cuda_error(void) { return g_cuda_error; }

}  // extern "C"
