/*
 * libdare — a stack of DARE attention layers inside pre-norm SwiGLU transformer blocks, with block-wise greedy
 * decoding: the setting DARE is plugged into (Sec. 3: "extends the standard diffusion inference pipeline";
 * Appendix A: block size 32, generation length 256).  The paper defines only the attention layer (Alg. 1, Alg. 2,
 * see dare.h); the block around it is read as
 *
 *     h   = x + DARE_attention(x)                       (dare_layer_step with the residual added)
 *     out = h + W_D ( silu(W_G n) * (W_U n) ),  n = RMSNorm_2(h)      (MLP on every active row, Appendix E.1)
 *
 * followed by a final RMSNorm and an untied LM head.  Decoding: the first step runs the whole sequence and fills
 * every cache; later steps run the generation window only (the prompt's K/V rows stay frozen: prefix cache); each
 * step un-masks, inside the active block, the masked position whose top-1 softmax probability is largest (lowest
 * index on ties), greedily; the mask token itself is never emitted.
 *
 * bf16 only, head_dim 128, d_model and vocab multiples of 256, d_ff a multiple of 128 (tensor-core kernels).
 * Same conventions as dare.h: device pointers unless named *_host, caller-owned workspace, status codes, work is
 * enqueued on the given stream.
 */
#ifndef DARE_STACK_H_
#define DARE_STACK_H_

#include "dare.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dare_stack dare_stack_t; /* opaque */

typedef struct {
  uint32_t struct_size;       /* sizeof(dare_stack_config_t) */
  int32_t n_layers;
  int32_t d_ff;               /* SwiGLU width */
  int32_t vocab;
  int32_t mask_id;            /* id of the mask token */
  int32_t block;              /* decoding block size (<= 32) */
  dare_layer_config_t layer;  /* geometry of every attention layer; max_seq = prompt + generation length */
} dare_stack_config_t;

typedef struct {
  dare_layer_weights_t attn;  /* W_Q, W_K, W_V, W_O, gain of the first norm */
  const float* gain2;         /* float32 [d_model], gain of the norm before the MLP */
  const void* w_gate;         /* [d_ff, d_model] */
  const void* w_up;           /* [d_ff, d_model] */
  const void* w_down;         /* [d_model, d_ff] */
} dare_block_weights_t;

typedef struct {
  const void* emb;                     /* [vocab, d_model] */
  const void* head;                    /* [vocab, d_model], untied */
  const float* final_gain;             /* float32 [d_model] */
  const dare_block_weights_t* blocks_host; /* HOST array of n_layers entries (device pointers inside) */
} dare_stack_weights_t;

size_t dare_stack_workspace_bytes(const dare_stack_config_t* cfg);
dare_status_t dare_stack_create(const dare_stack_config_t* cfg, const dare_stack_weights_t* weights, void* workspace,
                                size_t workspace_bytes, dare_stack_t** out);
dare_status_t dare_stack_reset(dare_stack_t* stack);
dare_status_t dare_stack_destroy(dare_stack_t* stack);

/* The handle of layer `index` (owned by the stack) for the observation calls of dare.h. */
dare_layer_t* dare_stack_layer(dare_stack_t* stack, int index);

/* One forward pass of the stack over positions [pos_begin, pos_begin + seq_act) of every sequence.
 *   tokens      int32 [batch, seq_total]: the full token buffer; the pass reads columns of the window
 *   taus_host   HOST float32 [n_layers]: threshold of every layer (Sec. 3.1: tau_l per layer)
 *   hidden_out  [batch, seq_act, d_model] bf16: the final-normed states (may be NULL)
 * State rules of every layer are those of dare_layer_step. */
dare_status_t dare_stack_forward(dare_stack_t* stack, const int32_t* tokens, int batch, int seq_total, int seq_act,
                                 int pos_begin, int mode, const float* taus_host, void* hidden_out, void* cuda_stream);

/* One decoding step: forward pass (whole sequence when `first`, else the window [prompt_len, seq_total)), logits of
 * the masked positions of block `block_index`, choice of (position, token) per sequence, and the write of the token
 * into `tokens`.
 *   forced_pos_host / forced_tok_host   HOST int32 [batch] or NULL: write these instead of the step's own choice
 *                                        (the step's own choice is still reported)
 *   pos_out / tok_out / prob_out        int32 / int32 / float32 [batch]: the step's own choice and its probability */
dare_status_t dare_stack_decode_step(dare_stack_t* stack, int32_t* tokens, int batch, int seq_total, int prompt_len,
                                     int block_index, int first, int mode, const float* taus_host,
                                     const int32_t* forced_pos_host, const int32_t* forced_tok_host, int32_t* pos_out,
                                     int32_t* tok_out, float* prob_out, void* cuda_stream);

/* Observation for tests: during every later pass, copy the input x and the output h = x + attention of layer
 * `layer_index` into the DEVICE buffers x_out / h_out ([batch, seq_act, d_model] bf16 each; NULL = skip;
 * layer_index < 0 switches the capture off). */
dare_status_t dare_stack_set_capture(dare_stack_t* stack, int layer_index, void* x_out, void* h_out);

/* Observation for tests: the final-normed hidden states [batch, seq_act, d_model] (bf16) of the last forward pass
 * or decoding step, copied to a HOST buffer of `bytes` bytes (synchronises the stream). */
dare_status_t dare_stack_last_hidden(dare_stack_t* stack, void* dst_host, size_t bytes, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* DARE_STACK_H_ */
