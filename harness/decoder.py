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
                 block, seed=0, flags=0, commit_mode="append"):
        """commit_mode "append": RoPE in torch, block K/V handed to the attention calls as tensors,
        accepted rows copied by orthrus_kv_append_layers.  "truncate": the projection outputs go
        through orthrus_rope_block_kv_write (rotation fused with the write of the block's K/V rows
        behind the prefix), the attention calls read the block from the cache, and the commit is
        orthrus_commit_len."""
        assert commit_mode in ("append", "truncate")
        self.commit_mode = commit_mode
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
        self._ws_by_block = {}
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

    def layer_objs(self, block, extra_flags=0):
        b = self.b
        hint = self.cap - block
        return [b.make_layer(self.k_cache[l], self.v_cache[l], self.cache_len, self.Hq, block, hint, 0.0,
                             self.flags | extra_flags) for l in range(self.L)]

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
    def forward_block(self, tokens, view, block, return_hidden=False, want_logits=True, record=None,
                      capture=None):
        """tokens [B][block] (id == vocab selects the mask embedding).  view 'diff' or 'ar'.
        Returns (logits [B][block][V], per-layer block K, per-layer block V), with
        return_hidden also the final-norm hidden states [B][block][H] the LM head is applied to.
        record: a list that receives one closure per library call (same arguments), so that a
        caller can replay the library's share of the pass on its own.
        capture: a dict {layer index: None}; the entry of each listed layer is replaced by the
        tensors of its attention call (q, k, v, out, cache_len; device clones), for parity checks."""
        b = self.b
        B = tokens.shape[0]
        h = self.emb[tokens.long()]
        pos = self.cache_len.long().unsqueeze(1) + torch.arange(block, device=h.device)
        truncate = self.commit_mode == "truncate"
        layers = self.layer_objs(block, b.LAYER_BLOCK_IN_CACHE if truncate else 0)
        # one workspace per block width, kept for good: captured graphs hold its address
        if block not in self._ws_by_block:
            self._ws_by_block[block] = b.new_workspace(b.orthrus_attend_workspace_bytes(layers[0]))
        self.ws = self._ws_by_block[block]
        sfx = "_d" if view == "diff" else ""
        ks, vs = [], []
        for l, lw in enumerate(self.layers):
            x = self.norm(h)
            fn = b.orthrus_diffusion_block_attend if view == "diff" else b.orthrus_ar_verify_attend
            if truncate:
                q_raw = (x @ lw["wq" + sfx]).view(B, block, self.Hq, self.d)
                k = (x @ lw["wk" + sfx]).view(B, block, self.Hkv, self.d)
                v = (x @ lw["wv" + sfx]).view(B, block, self.Hkv, self.d)
                q = torch.empty_like(q_raw)
                out = torch.empty_like(q)
                call = (lambda fn=fn, L=layers[l], q_raw=q_raw, q=q, k=k, v=v, out=out, ws=self.ws:
                        (b.orthrus_rope_block_kv_write(L, q_raw, k, v, 10000.0, q, ws),
                         fn(L, q, None, None, out, ws)))
            else:
                q = self.rope((x @ lw["wq" + sfx]).view(B, block, self.Hq, self.d), pos).contiguous()
                k = self.rope((x @ lw["wk" + sfx]).view(B, block, self.Hkv, self.d), pos).contiguous()
                v = (x @ lw["wv" + sfx]).view(B, block, self.Hkv, self.d).contiguous()
                out = torch.empty_like(q)
                call = (lambda fn=fn, L=layers[l], q=q, k=k, v=v, out=out, ws=self.ws: fn(L, q, k, v, out, ws))
            call()
            if capture is not None and l in capture:
                capture[l] = dict(q=q.clone(), k=k.clone(), v=v.clone(), out=out.clone(),
                                  cache_len=self.cache_len.clone())
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
        if self.commit_mode == "truncate":
            # the AR pass left its block rows behind the prefix of every layer: only the length moves
            self.b.orthrus_commit_len(self.layer_objs(block)[0], n_commit, self.ws)
        else:
            self.b.orthrus_kv_append_layers(self.layer_objs(block), ks, vs, n_commit, True, self.ws)

    def status(self):
        """OR of the device status words of every workspace this decoder has used."""
        st = 0
        for ws in self._ws_by_block.values():
            st |= self.b.orthrus_read_status(ws)
        return st


class ForcedDraftLoop:
    """The generation loop of Section 3.3 on a Decoder, with the diffusion view's drafts replaced by
    forced ones so that acceptance is controlled (a random-initialised diffusion head proposes
    nothing useful; its pass still runs in full).

    Every cycle first looks ahead: `block` width-1 greedy steps of the AR view through the same
    library calls give the tokens plain autoregressive decoding would emit next from the
    current state; the cache length is then rewound (the rows the look-ahead wrote lie behind
    it and are overwritten by the cycle's own commit).  Draft i is look-ahead token i with
    probability `rate`, else a uniform token.  The look-ahead is also the reference of the
    lossless check: the tokens a cycle commits must be its first n look-ahead tokens.  Because the
    reference restarts from the loop's own state every cycle, a near-tie that block verification
    and width-1 decoding round differently costs one mismatch and nothing after it."""

    def __init__(self, dec, anchor, rate, seed=0, fused=True):
        self.dec, self.rate, self.fused = dec, rate, fused
        b, B, K, V = dec.b, dec.B, dec.K, dec.V
        dev = anchor.device
        i32 = dict(dtype=torch.int32, device=dev)
        self.anchor = anchor.clone()
        self.anchor1 = anchor.clone()
        self.draft = torch.zeros(B, K, **i32)
        self.look = torch.zeros(B, K, **i32)
        self.gaps = torch.zeros(B, K, dtype=torch.float32, device=dev)
        self.done = torch.zeros(B, dtype=torch.int64, device=dev)
        self.outs1 = [torch.zeros(B, **i32), torch.zeros(B, 1, **i32), torch.zeros(B, 1, **i32),
                      torch.zeros(B, **i32)]
        self.zero1 = torch.zeros(B, 1, **i32)
        self.ws1 = b.new_workspace(b.orthrus_lm_head_consensus_workspace_bytes(B, 1, V), device=dev)
        self.wsK = b.new_workspace(b.orthrus_lm_head_consensus_workspace_bytes(B, K, V), device=dev)
        self.cws1 = b.new_workspace(b.orthrus_consensus_workspace_bytes(B, 1, V), device=dev)
        self.gen = torch.Generator(device=dev)
        self.gen.manual_seed(seed)
        self.len_saved = dec.cache_len.clone()
        self.logits = None            # AR logits of the last cycle (two-step consensus only)

    # ---- width-1 reference steps
    def k1_step(self, j, want_gap=False):
        dec, b = self.dec, self.dec.b
        logits, ks, vs, hn = dec.forward_block(self.anchor1.view(-1, 1), "ar", 1, return_hidden=True,
                                               want_logits=want_gap or not self.fused)
        if self.fused:
            b.orthrus_lm_head_consensus(hn, dec.lm_head_rows(), self.zero1, *self.outs1, self.ws1)
        else:
            b.orthrus_consensus_accept(logits, self.zero1, *self.outs1, self.cws1)
        if want_gap:
            top2 = logits.float().topk(2, dim=-1).values[:, 0]
            self.gaps[:, j] = top2[:, 0] - top2[:, 1]
        dec.commit(ks, vs, self.outs1[0], 1)
        self.anchor1.copy_(self.outs1[3])
        self.look[:, j] = self.outs1[3]

    def lookahead(self, want_gap=False):
        dec = self.dec
        self.len_saved.copy_(dec.cache_len)
        self.anchor1.copy_(self.anchor)
        for j in range(dec.K):
            self.k1_step(j, want_gap)
        dec.cache_len.copy_(self.len_saved)

    def force_drafts(self):
        B, K, V = self.dec.B, self.dec.K, self.dec.V
        dev = self.draft.device
        coin = torch.rand(B, K, device=dev, generator=self.gen) < self.rate
        rnd = torch.randint(0, V, (B, K), device=dev, generator=self.gen, dtype=torch.int32)
        self.draft.copy_(torch.where(coin, self.look, rnd))

    # ---- one cycle: both passes, the consensus, the commit
    def cycle(self, record=None, capture_diff=None, capture_ar=None):
        dec, b = self.dec, self.dec.b
        B, K, V = dec.B, dec.K, dec.V
        blk = torch.full((B, K), V, dtype=torch.int32, device=self.draft.device)
        blk[:, 0] = self.anchor
        dec.forward_block(blk, "diff", K, want_logits=False, record=record, capture=capture_diff)
        ar_in = torch.cat([self.anchor.view(B, 1), self.draft[:, :K - 1]], dim=1)
        logits, ks, vs, hn = dec.forward_block(ar_in, "ar", K, return_hidden=True, want_logits=not self.fused,
                                               record=record, capture=capture_ar)
        self.logits = logits
        if self.fused:
            tail = (lambda: (b.orthrus_lm_head_consensus(hn, dec.lm_head_rows(), self.draft, dec.n_commit,
                                                         dec.committed, dec.ar_argmax, dec.next_anchor, self.wsK),
                             dec.commit(ks, vs, dec.n_commit, K)))
        else:
            tail = (lambda: (b.orthrus_consensus_accept(logits, self.draft, dec.n_commit, dec.committed,
                                                        dec.ar_argmax, dec.next_anchor, dec.cws),
                             dec.commit(ks, vs, dec.n_commit, K)))
        tail()
        if record is not None:
            record.append(tail)
        self.done.add_(dec.n_commit.long())
        self.anchor.copy_(dec.next_anchor)

    def status(self):
        b = self.dec.b
        return self.dec.status() | b.orthrus_read_status(self.ws1) | b.orthrus_read_status(self.wsK)
