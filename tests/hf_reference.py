"""An independent library implementation of the Llama decoder (HuggingFace
transformers, CPU, float64) loaded with the same bf16 weights.  The paper's own
implementation is built on this architecture (Section 4 "Setup"), so the oracle's
special cases must reduce to it.  Used only to pin the oracle."""
import numpy as np
import torch

import synth_inputs as si


def build_hf_llama(shape, weights):
    from transformers import LlamaConfig, LlamaForCausalLM
    s = shape
    cfg = LlamaConfig(hidden_size=s.d, intermediate_size=s.F, num_hidden_layers=s.L, num_attention_heads=s.H,
                      num_key_value_heads=s.Hkv, vocab_size=s.V, rms_norm_eps=s.eps, rope_theta=s.theta,
                      tie_word_embeddings=False, head_dim=s.dh, max_position_embeddings=4096,
                      attention_bias=False, mlp_bias=False)
    cfg._attn_implementation = "eager"
    model = LlamaForCausalLM(cfg).double().eval()

    def f(bits):
        return torch.from_numpy(si.bf16_bits_to_f32(np.ascontiguousarray(bits)).astype(np.float64))

    sd = {"model.embed_tokens.weight": f(weights["embed"]), "lm_head.weight": f(weights["lm_head"]),
          "model.norm.weight": f(weights["g_final"])}
    for i, lw in enumerate(weights["layers"]):
        p = "model.layers.%d." % i
        sd[p + "self_attn.q_proj.weight"] = f(lw["wqkv"][: s.n_q])
        sd[p + "self_attn.k_proj.weight"] = f(lw["wqkv"][s.n_q: s.n_q + s.n_kv])
        sd[p + "self_attn.v_proj.weight"] = f(lw["wqkv"][s.n_q + s.n_kv:])
        sd[p + "self_attn.o_proj.weight"] = f(lw["wo"])
        sd[p + "mlp.gate_proj.weight"] = f(lw["wgu"][: s.F])
        sd[p + "mlp.up_proj.weight"] = f(lw["wgu"][s.F:])
        sd[p + "mlp.down_proj.weight"] = f(lw["wd"])
        sd[p + "input_layernorm.weight"] = f(lw["g_attn"])
        sd[p + "post_attention_layernorm.weight"] = f(lw["g_mlp"])
    model.load_state_dict(sd, strict=True)
    return model


def hf_logits(model, token_ids, visible=None):
    """Causal forward, no cache: logits [len, V] as float64 numpy.  visible: optional [len, len] 0/1
    matrix replacing the causal mask (row r attends to column c iff visible[r, c])."""
    with torch.no_grad():
        ids = torch.as_tensor(np.asarray(token_ids, dtype=np.int64))[None]
        mask = None
        if visible is not None:
            vis = torch.as_tensor(np.asarray(visible, dtype=bool))
            mask = torch.zeros(vis.shape, dtype=torch.float64).masked_fill(~vis, float("-inf"))[None, None]
        return model(ids, attention_mask=mask, use_cache=False).logits[0].numpy()


def hf_greedy(model, prompt_ids, count):
    """Cache-free greedy decoding by full recompute."""
    ids = [int(t) for t in prompt_ids]
    out = []
    for _ in range(count):
        t = int(np.argmax(hf_logits(model, ids)[-1]))
        out.append(t)
        ids.append(t)
    return out


def hf_kv(model, token_ids):
    """Post-rotary keys and values of a from-scratch forward: lists per layer of [len, Hkv*dh]."""
    with torch.no_grad():
        ids = torch.as_tensor(np.asarray(token_ids, dtype=np.int64))[None]
        out = model(ids, use_cache=True)
    pkv = out.past_key_values
    ks, vs = [], []
    for layer in range(model.config.num_hidden_layers):
        try:
            k, v = pkv.layers[layer].keys, pkv.layers[layer].values
        except AttributeError:
            k, v = pkv[layer][0], pkv[layer][1]
        ks.append(k[0].transpose(0, 1).reshape(k.shape[2], -1).numpy())
        vs.append(v[0].transpose(0, 1).reshape(v.shape[2], -1).numpy())
    return ks, vs


def hf_logits_with_replaced_rows(model, token_ids, layer, first_row, maps_w, maps_b, anchor_row, visible=None,
                                 prenorm=False):
    """Causal forward in which, at the input of decoder layer `layer`, rows
    first_row.. are replaced by W_i h[anchor_row] + b_i (i = 0..len(maps_w)-1).
    `layer` may be a sequence with one layer per row: row first_row + i is then
    replaced at the input of layer[i] (what it held before is never read by a row
    that matters, because the sequence is causal and the layers do not decrease).
    prenorm: the maps read the anchor row through that layer's own input RMSNorm module."""
    layers = [int(layer)] * len(maps_w) if np.isscalar(layer) else [int(t) for t in layer]
    assert len(layers) == len(maps_w) and layers == sorted(layers)

    def make_hook(at):
        def hook(module, args, kwargs):
            hs = args[0] if args else kwargs["hidden_states"]
            hs = hs.clone()
            src = hs[0, anchor_row]
            if prenorm:
                src = module.input_layernorm(src[None])[0]
            for i, W in enumerate(maps_w):
                if layers[i] == at:
                    hs[0, first_row + i] = torch.from_numpy(W) @ src + torch.from_numpy(maps_b[i])
            if args:
                return (hs,) + tuple(args[1:]), kwargs
            kwargs = dict(kwargs)
            kwargs["hidden_states"] = hs
            return args, kwargs
        return hook

    handles = [model.model.layers[at].register_forward_pre_hook(make_hook(at), with_kwargs=True) for at in sorted(set(layers))]
    try:
        return hf_logits(model, token_ids, visible)
    finally:
        for h in handles:
            h.remove()
