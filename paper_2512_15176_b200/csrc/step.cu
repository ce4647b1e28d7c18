// One greedy verify step driven from host buffers: the end-to-end form of
// Algorithm 1's loop body on the verifier side (copy the block in, score it,
// accept, commit, copy the verdict out).

#include "common.cuh"

extern "C" int deer_verify_step_host(deer_kv* kv, const deer_step_dev* dev, const void* w, const void* q_host,
                                     const void* k_blk_host, const void* v_blk_host, const void* h_host,
                                     const int32_t* draft_ids_host, int B, int k, int Hq, int hid, int V, float scale,
                                     int max_seq_len, int32_t* accept_len_host, int32_t* out_ids_host, int32_t* n_out_host,
                                     void* stream) {
    DEER_CHECK_ARG(kv && dev && w && q_host && k_blk_host && v_blk_host && h_host && draft_ids_host && accept_len_host &&
                       out_ids_host && n_out_host,
                   DEER_ERR_INVALID_ARG, "deer_verify_step_host: null argument");
    DEER_CHECK_ARG(B > 0 && k >= 1 && k <= DEER_MAX_BLOCK, DEER_ERR_UNSUPPORTED, "deer_verify_step_host: bad B or k");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int Hkv = kv->d.n_kv_heads, D = kv->d.head_dim;
    const size_t M = (size_t)B * k;
    DEER_CUDA(cudaMemcpyAsync(dev->q, q_host, M * Hq * D * 2, cudaMemcpyHostToDevice, st));
    DEER_CUDA(cudaMemcpyAsync(dev->k_blk, k_blk_host, M * Hkv * D * 2, cudaMemcpyHostToDevice, st));
    DEER_CUDA(cudaMemcpyAsync(dev->v_blk, v_blk_host, M * Hkv * D * 2, cudaMemcpyHostToDevice, st));
    DEER_CUDA(cudaMemcpyAsync(dev->h, h_host, M * hid * 2, cudaMemcpyHostToDevice, st));
    DEER_CUDA(cudaMemcpyAsync(dev->draft_ids, draft_ids_host, M * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    int rc = deer_kv_reserve(kv, dev->seq_ids, B, k, stream);
    if (rc != DEER_OK) return rc;
    rc = deer_block_attn(kv, dev->seq_ids, dev->q, dev->k_blk, dev->v_blk, dev->attn_out, B, k, Hq, DEER_MASK_CAUSAL, 1, scale,
                         max_seq_len, dev->attn_ws, dev->attn_ws_bytes, stream);
    if (rc != DEER_OK) return rc;
    rc = deer_lmhead_select(dev->h, w, (int)M, hid, V, DEER_SEL_ARGMAX, 1.f, nullptr, dev->target_ids, nullptr, nullptr, nullptr,
                            nullptr, dev->lm_ws, dev->lm_ws_bytes, stream);
    if (rc != DEER_OK) return rc;
    rc = deer_accept(DEER_ACC_GREEDY, B, k, V, dev->draft_ids, dev->target_ids, nullptr, nullptr, nullptr, 1.f, nullptr, nullptr,
                     nullptr, -1, dev->accept_len, dev->out_ids, dev->n_out, nullptr, 0, stream);
    if (rc != DEER_OK) return rc;
    rc = deer_kv_commit(kv, dev->seq_ids, dev->accept_len, B, k, stream);
    if (rc != DEER_OK) return rc;
    DEER_CUDA(cudaMemcpyAsync(accept_len_host, dev->accept_len, (size_t)B * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    DEER_CUDA(cudaMemcpyAsync(out_ids_host, dev->out_ids, M * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    DEER_CUDA(cudaMemcpyAsync(n_out_host, dev->n_out, (size_t)B * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    DEER_CUDA(cudaStreamSynchronize(st));
    return DEER_OK;
}
