"""CPU oracle for the LoMA hot path (test infrastructure, not product code).

Everything under this package is a plain, slow, fp64 NumPy restatement of what
the paper defines: the chunk layout (Section 4.1), the attention mask
(Eq. 1-3), masked softmax attention (Eq. 6-7) and its gradients (Section 4.4), and the generation-time cache
algebra (Section 3.1 and Appendix A).  It exists only so that tests, the smoke
check and the CPU-baseline leg of the benchmark have something independent to
compare the CUDA library against.  It shares no code with the CUDA path and the
CUDA path never calls it.
"""

from .loma_oracle import (  # noqa: F401
    FLAG_MEM_SEES_PRIOR_MEM,
    FLAG_NO_REP_ZONE,
    ZONE_READ,
    ZONE_MEM,
    ZONE_REP,
    chunk_len,
    seq_len,
    decompose,
    layout_index,
    generation_index,
    allowed,
    chunk_mask,
    cross_chunk_block,
    dense_mask,
    mask_rows,
    masked_softmax_attention,
    masked_attn_fwd,
    masked_softmax_attention_bwd,
    masked_attn_bwd,
    masked_attn_bwd_dq_rows,
    masked_attn_bwd_dkv_cols,
    position_ids,
    rope_rotate,
    rope_apply,
    decode_attn,
    prefill_attn,
    replay_prompt_pieces,
    decode_attn_ragged,
    decode_attn_paged,
    paged_to_contiguous,
    compress_step,
    compress_step_ragged,
    compress_step_paged,
    replay_generation,
)
