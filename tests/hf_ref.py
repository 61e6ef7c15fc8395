"""An independent Llama implementation (HuggingFace transformers, CPU fp32) loaded with the synthetic
weights.  Used only to pin the CPU oracle: it shares no code with the oracle or the CUDA path."""
import torch
from transformers import LlamaConfig, LlamaForCausalLM


def _cfg(cfg, n_layers, vocab):
    return LlamaConfig(vocab_size=vocab, hidden_size=cfg.hidden, intermediate_size=cfg.ffn,
                       num_hidden_layers=n_layers, num_attention_heads=cfg.n_heads,
                       num_key_value_heads=cfg.n_kv_heads, head_dim=cfg.head_dim, rms_norm_eps=cfg.rms_eps,
                       rope_theta=cfg.rope_theta, max_position_embeddings=1 << 15, attention_bias=False,
                       mlp_bias=False, tie_word_embeddings=False, attn_implementation="eager")


_MAP = {"attn_norm": "input_layernorm.weight", "wq": "self_attn.q_proj.weight", "wk": "self_attn.k_proj.weight",
        "wv": "self_attn.v_proj.weight", "wo": "self_attn.o_proj.weight",
        "mlp_norm": "post_attention_layernorm.weight", "w_gate": "mlp.gate_proj.weight",
        "w_up": "mlp.up_proj.weight", "w_down": "mlp.down_proj.weight"}


def _load(model, embed, final_norm, lm_head, layers):
    sd = {"model.embed_tokens.weight": embed, "model.norm.weight": final_norm, "lm_head.weight": lm_head}
    for i, l in enumerate(layers):
        for k, v in _MAP.items():
            sd[f"model.layers.{i}.{v}"] = l[k]
    sd = {k: v.to(torch.float32) for k, v in sd.items()}
    missing, unexpected = model.load_state_dict(sd, strict=False)
    assert not [m for m in missing if "rotary" not in m], missing
    assert not unexpected, unexpected
    return model.eval()


def target_model(cfg, tw):
    m = LlamaForCausalLM(_cfg(cfg, cfg.n_layers, cfg.vocab))
    return _load(m, tw["embed"], tw["final_norm"], tw["lm_head"], tw["layers"])


def draft_model(cfg, dw):
    """The draft's decoder layer + norm + reduced-vocabulary head; feed it `inputs_embeds`."""
    m = LlamaForCausalLM(_cfg(cfg, 1, cfg.draft_vocab))
    emb = torch.zeros(cfg.draft_vocab, cfg.hidden)
    return _load(m, emb, dw["final_norm"], dw["lm_head"], [dw])


class BlockOutputs:
    """Captures the residual stream after every decoder block (before the final norm)."""

    def __init__(self, model):
        self.outs = []
        self.hooks = [l.register_forward_hook(self._hook) for l in model.model.layers]

    def _hook(self, mod, inp, out):
        self.outs.append((out[0] if isinstance(out, tuple) else out).detach())

    def close(self):
        for h in self.hooks:
            h.remove()


@torch.no_grad()
def forward(model, ids=None, embeds=None, position_ids=None, mask_bool=None):
    """Returns (logits [T,V], [residual after block l] list of [T,k]).  mask_bool: [T,T] visibility."""
    cap = BlockOutputs(model)
    kw = {}
    if mask_bool is not None:
        m = torch.zeros(mask_bool.shape, dtype=torch.float32)
        m[~mask_bool] = torch.finfo(torch.float32).min
        kw["attention_mask"] = m[None, None]
    if position_ids is not None:
        kw["position_ids"] = position_ids[None]
    if ids is not None:
        out = model(input_ids=ids[None].long(), use_cache=False, **kw)
    else:
        out = model(inputs_embeds=embeds[None], use_cache=False, **kw)
    cap.close()
    return out.logits[0], [o[0] if o.dim() == 3 else o for o in cap.outs]
