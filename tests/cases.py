"""Small model variants shared by the test modules (inputs only; built from synth.Config)."""
import synth

TINY = synth.CONFIGS["tiny"]
# grouped-query attention, non-unit norm gains, depth-decaying branches, 6 layers: has rejections
TINY_GQA = synth.small_variant(TINY, name="tiny_gqa", n_layers=6, n_kv_heads=2, gain_spread=0.1,
                               residual_scaling="decay", e_min=1, e_max=5, g_max=5, emb_scale=10.0,
                               prompt_len=40, gen_len=48, seed=77)
# ragged shapes: prompt shorter than the initialisation window, odd generation length
# long prompts: the bulk of the prompt goes through the tensor-core prefill (ragged last row tile)
TINY_LONG = synth.small_variant(TINY, name="tiny_long", prompt_len=300, gen_len=24, emb_scale=10.0, seed=11)
TINY_GQA_LONG = synth.small_variant(TINY_GQA, name="tiny_gqa_long", prompt_len=200, gen_len=24, seed=78)
# two prefill passes of 512 positions; in the second variant the 32-position window straddles the pass boundary
TINY_LONG2 = synth.small_variant(TINY, name="tiny_long2", prompt_len=600, gen_len=16, emb_scale=10.0, seed=12)
TINY_LONG3 = synth.small_variant(TINY_GQA, name="tiny_gqa_long3", prompt_len=530, gen_len=16, seed=79)
TINY_SHORT = synth.small_variant(TINY, name="tiny_short", prompt_len=7, gen_len=21, emb_scale=10.0, seed=5)
# head dimension 128 (the shape the tcgen05 prefill attention serves): a ragged last query tile; and two prefill passes
# with grouped-query attention
TINY_HD128 = synth.small_variant(TINY, name="tiny_hd128", n_heads=2, n_kv_heads=2, head_dim=128, prompt_len=300, gen_len=24,
                                 emb_scale=10.0, seed=21)
TINY_HD128_GQA = synth.small_variant(TINY_GQA, name="tiny_hd128_gqa", n_heads=4, n_kv_heads=2, head_dim=128, prompt_len=600,
                                     gen_len=16, seed=22)
