"""The HuggingFace Llama implementation (the one the paper patched) loaded with
the synthetic weights, in fp64 on the CPU: an independent restatement of the
decoder block that the oracle is pinned to."""
import contextlib

import torch


def build(shape, w, max_pos=512):
    from transformers import LlamaConfig, LlamaForCausalLM
    cfg = LlamaConfig(vocab_size=shape.vocab, hidden_size=shape.d_model,
                      intermediate_size=shape.d_ffn, num_hidden_layers=shape.n_layers,
                      num_attention_heads=shape.n_q_heads, num_key_value_heads=shape.n_kv_heads,
                      head_dim=shape.head_dim, rms_norm_eps=shape.rms_eps,
                      rope_theta=shape.rope_base, attention_bias=False, mlp_bias=False,
                      tie_word_embeddings=False, max_position_embeddings=max_pos,
                      attn_implementation="eager")
    m = LlamaForCausalLM(cfg).to(torch.float64).eval()
    nq = shape.n_q_heads * shape.head_dim
    nkv = shape.n_kv_heads * shape.head_dim
    with torch.no_grad():
        m.model.embed_tokens.weight.copy_(w["embed"].double())
        m.lm_head.weight.copy_(w["lm_head"].double())
        m.model.norm.weight.copy_(w["final_norm"].double())
        for l, lay in enumerate(m.model.layers):
            lay.input_layernorm.weight.copy_(w["attn_norm"][l].double())
            lay.post_attention_layernorm.weight.copy_(w["mlp_norm"][l].double())
            lay.self_attn.q_proj.weight.copy_(w["wqkv"][l][:nq].double())
            lay.self_attn.k_proj.weight.copy_(w["wqkv"][l][nq:nq + nkv].double())
            lay.self_attn.v_proj.weight.copy_(w["wqkv"][l][nq + nkv:].double())
            lay.self_attn.o_proj.weight.copy_(w["wo"][l].double())
            lay.mlp.gate_proj.weight.copy_(w["w_gate"][l].double())
            lay.mlp.up_proj.weight.copy_(w["w_up"][l].double())
            lay.mlp.down_proj.weight.copy_(w["w_down"][l].double())
    return m, cfg


@contextlib.contextmanager
def only_layers(model, keep):
    """The model with every decoder layer outside `keep` deleted (each kept layer
    still addresses its own entry of the KV cache)."""
    full = model.model.layers
    n_full = model.config.num_hidden_layers
    model.model.layers = torch.nn.ModuleList([full[i] for i in keep])
    model.config.num_hidden_layers = len(keep)
    try:
        yield model
    finally:
        model.model.layers = full
        model.config.num_hidden_layers = n_full
