"""A random-initialised decoder around the library calls, for the generation-loop tests and
the benchmark's whole-cycle timing.

Harness only, not part of the library's path.  Everything off the hot path (embeddings, RMSNorm, RoPE, the Q/K/V/O
projections of both views, the SwiGLU FFN, the LM head) is plain torch; the four steps of
the hot path go through the C ABI: orthrus_diffusion_block_attend, orthrus_ar_verify_attend,
orthrus_consensus_accept (or orthrus_lm_head_consensus) and orthrus_kv_append_layers.  Only the diffusion view's Q/K/V
projections are separate weights; output projection, FFN, norms, embeddings and LM head are
shared with the AR view (Section 3.1).  The block is the anchor followed by K-1 copies of a
mask embedding (Section 3.3); block position i has rotary position P_b + i.
"""
import math

import torch


class Decoder:
    def __init__(self, binding, layers, hidden, n_q, n_kv, d, ffn, vocab, dtype, batch, capacity,
                 block, seed=0, flags=0):
        self.b, self.L, self.H, self.Hq, self.Hkv, self.d = binding, layers, hidden, n_q, n_kv, d
        self.V, self.dtype, self.B, self.cap, self.K = vocab, dtype, batch, capacity, block
        g = torch.Generator().manual_seed(seed)
        dev = "cuda"

        def w(*shape, std=0.02):
            return (torch.randn(*shape, generator=g) * std).to(dtype).to(dev)

        self.emb = w(vocab + 1, hidden, std=1.0)          # row `vocab` is the mask embedding
        self.lm_head = w(hidden, vocab, std=1.0 / math.sqrt(hidden))
        s = 1.0 / math.sqrt(hidden)
        self.layers = []
        for _ in range(layers):
            lw = dict(wq=w(hidden, n_q * d, std=s), wk=w(hidden, n_kv * d, std=s), wv=w(hidden, n_kv * d, std=s),
                      wo=w(n_q * d, hidden, std=1.0 / math.sqrt(n_q * d)),
                      w1=w(hidden, ffn, std=s), w3=w(hidden, ffn, std=s), w2=w(ffn, hidden, std=1.0 / math.sqrt(ffn)))
            # the diffusion projections start from the AR ones (Section 3.1) and drift a little
            for n in ("wq", "wk", "wv"):
                lw[n + "_d"] = (lw[n].float() + 0.1 * s * torch.randn(lw[n].shape, generator=g).to(dev)).to(dtype)
            self.layers.append(lw)
        self.k_cache = [torch.zeros(batch, n_kv, capacity, d, dtype=dtype, device=dev) for _ in range(layers)]
        self.v_cache = [torch.zeros(batch, n_kv, capacity, d, dtype=dtype, device=dev) for _ in range(layers)]
        self.cache_len = torch.zeros(batch, dtype=torch.int32, device=dev)
        self.flags = flags
        self.ws = None
        self.cws = binding.new_workspace(binding.orthrus_consensus_workspace_bytes(batch, block, vocab))
        i32 = dict(dtype=torch.int32, device=dev)
        self.n_commit = torch.zeros(batch, **i32)
        self.committed = torch.zeros(batch, block, **i32)
        self.ar_argmax = torch.zeros(batch, block, **i32)
        self.next_anchor = torch.zeros(batch, **i32)

    # ------------------------------------------------------------------ torch-side pieces
    @staticmethod
    def norm(x):
        xf = x.float()
        return (xf * torch.rsqrt(xf.pow(2).mean(-1, keepdim=True) + 1e-6)).to(x.dtype)

    def rope(self, x, pos):
        """x [B][T][heads][d], pos [B][T] (absolute positions)."""
        half = self.d // 2
        inv = 1.0 / (10000.0 ** (torch.arange(half, device=x.device, dtype=torch.float32) / half))
        ang = pos.float().unsqueeze(-1) * inv                      # [B][T][half]
        c, s = ang.cos().unsqueeze(2), ang.sin().unsqueeze(2)
        xf = x.float()
        a, b_ = xf[..., :half], xf[..., half:]
        return torch.cat([a * c - b_ * s, a * s + b_ * c], dim=-1).to(x.dtype)

    def ffn(self, lw, h):
        x = self.norm(h)
        return h + (torch.nn.functional.silu(x @ lw["w1"]) * (x @ lw["w3"])) @ lw["w2"]

    def layer_objs(self, block):
        b = self.b
        hint = self.cap - block
        return [b.make_layer(self.k_cache[l], self.v_cache[l], self.cache_len, self.Hq, block, hint, 0.0,
                             self.flags) for l in range(self.L)]

    # ------------------------------------------------------------------ prefill (torch)
    def prefill(self, prompt):
        """Causal forward over the prompt [B][T]; fills the caches with positions 0..T-2 and
        returns the last prompt token as the first anchor (its KV comes from the block)."""
        B, T = prompt.shape
        h = self.emb[prompt.long()]
        pos = torch.arange(T, device=h.device).expand(B, T)
        G = self.Hq // self.Hkv
        for l, lw in enumerate(self.layers):
            x = self.norm(h)
            q = self.rope((x @ lw["wq"]).view(B, T, self.Hq, self.d), pos)
            k = self.rope((x @ lw["wk"]).view(B, T, self.Hkv, self.d), pos)
            v = (x @ lw["wv"]).view(B, T, self.Hkv, self.d)
            self.k_cache[l][:, :, :T - 1] = k[:, :T - 1].transpose(1, 2)
            self.v_cache[l][:, :, :T - 1] = v[:, :T - 1].transpose(1, 2)
            kk = k.transpose(1, 2).repeat_interleave(G, dim=1).float()
            vv = v.transpose(1, 2).repeat_interleave(G, dim=1).float()
            o = torch.nn.functional.scaled_dot_product_attention(q.transpose(1, 2).float(), kk, vv, is_causal=True)
            h = h + o.transpose(1, 2).reshape(B, T, self.Hq * self.d).to(h.dtype) @ lw["wo"]
            h = self.ffn(lw, h)
        self.cache_len.fill_(T - 1)
        return prompt[:, -1].to(torch.int32)

    # ------------------------------------------------------------------ one pass through the layers
    def forward_block(self, tokens, view, block, return_hidden=False, want_logits=True, record=None):
        """tokens [B][block] (id == vocab selects the mask embedding).  view 'diff' or 'ar'.
        Returns (logits [B][block][V], per-layer block K, per-layer block V), with
        return_hidden also the final-norm hidden states [B][block][H] the LM head is applied to.
        record: a list that receives one closure per library call (same arguments), so that a
        caller can replay the library's share of the pass on its own."""
        b = self.b
        B = tokens.shape[0]
        h = self.emb[tokens.long()]
        pos = self.cache_len.long().unsqueeze(1) + torch.arange(block, device=h.device)
        layers = self.layer_objs(block)
        if self.ws is None or self.ws_block != block:
            self.ws = b.new_workspace(b.orthrus_attend_workspace_bytes(layers[0]))
            self.ws_block = block
        sfx = "_d" if view == "diff" else ""
        ks, vs = [], []
        for l, lw in enumerate(self.layers):
            x = self.norm(h)
            q = self.rope((x @ lw["wq" + sfx]).view(B, block, self.Hq, self.d), pos).contiguous()
            k = self.rope((x @ lw["wk" + sfx]).view(B, block, self.Hkv, self.d), pos).contiguous()
            v = (x @ lw["wv" + sfx]).view(B, block, self.Hkv, self.d).contiguous()
            out = torch.empty_like(q)
            fn = b.orthrus_diffusion_block_attend if view == "diff" else b.orthrus_ar_verify_attend
            call = (lambda fn=fn, L=layers[l], q=q, k=k, v=v, out=out: fn(L, q, k, v, out, self.ws))
            call()
            if record is not None:
                record.append(call)
            h = h + out.view(B, block, self.Hq * self.d) @ lw["wo"]
            h = self.ffn(lw, h)
            ks.append(k); vs.append(v)
        hn = self.norm(h).contiguous()
        logits = (hn @ self.lm_head).contiguous() if want_logits else None
        if return_hidden:
            return logits, ks, vs, hn
        return logits, ks, vs

    def lm_head_rows(self):
        """The LM head as [V][H] rows, the layout orthrus_lm_head_consensus takes."""
        if not hasattr(self, "_lm_head_rows"):
            self._lm_head_rows = self.lm_head.t().contiguous()
        return self._lm_head_rows

    def commit(self, ks, vs, n_commit, block):
        self.b.orthrus_kv_append_layers(self.layer_objs(block), ks, vs, n_commit, True, self.ws)
