"""Buffers and call sequences of the benchmark/parity workloads, over the ``api`` binding.

Only plumbing lives here: tensors are allocated and filled from the seeded generators, host offset
tables are laid out, and the library's entry points are called in the order the path prescribes
(score+select -> gather -> attend per decode token).  The benchmark and the full-size parity tests
both drive the GPU through this module, so what is timed is what is checked.
"""
from __future__ import annotations

import numpy as np
import torch

from . import inputs
from .inputs import Workload


class CompressDecode:
    """One layer instance: compress each sequence's context at ratio r, then decode token by token.

    Layout (all packed, row = one token's H*dh elements):
      X, K, V      [sum n_b, ...]   context hidden states and their K/V rows
      cacheK/V     [sum cap_b, ...] nugget cache, region b starts at cache_off[b]
      locK/V       [B * (local + tq + steps), ...] uncompressed tokens after the context: `local`
                   context tokens, then the `tq` tokens of the query block, then the decoded tokens,
                   at consecutive positions from n_b on
      Qb, Ob       [B * tq, H, dh] the query block (compressor mode, Eq. 13): token i of sequence b
                   sits at position n_b + local + i and sees the nuggets, the local context and,
                   causally, the block itself
      Qd           [steps, B, H, dh] decode queries;  Od the same shape, written by attend.  Decode
                   token s sits at position n_b + local + tq + s.  With `sliding` the window is the
                   `local` most recent positions including the token itself (rows [s+1, s+1+local));
                   otherwise nothing is evicted and the window is rows [0, local + tq + s + 1)
    """

    def __init__(self, dodo, wl: Workload, r: int, tag, gen_device="cuda", steps: int | None = None,
                 sliding: bool | None = None, with_lse: bool = False):
        self.dodo, self.wl, self.r = dodo, wl, r
        self.steps = wl.decode_steps if steps is None else steps
        self.tq = wl.tq_dense
        # a sliding window only makes sense when the window is seeded and no query block precedes it
        self.sliding = (wl.local > 0 and wl.tq_dense == 0) if sliding is None else sliding
        B, H, dh, d = wl.B, wl.H, wl.dh, wl.d
        dt = wl.dtype
        self.n = np.asarray(wl.n_ctx, dtype=np.int32)
        self.seq_off = inputs.offsets(self.n)
        self.k = np.asarray([dodo.num_nuggets(int(n), r) for n in self.n], dtype=np.int32)
        self.nug_off = inputs.offsets(self.k)
        self.cache_off = inputs.offsets(self.k)
        N, Kt = int(self.seq_off[-1]), int(self.nug_off[-1])

        def draw(shape, name, std=1.0, dtype=dt):
            return inputs.randn(shape, *tag, name, std=std, dtype=dtype, device=gen_device).cuda()

        self.X = draw((N, d), "X")
        self.w = draw((d,), "w", std=d ** -0.5)
        if wl.project_kv:
            Xh = self.X.cpu()
            Wk = inputs.randn((d, H * dh), *tag, "Wk", std=d ** -0.5, dtype=dt)
            Wv = inputs.randn((d, H * dh), *tag, "Wv", std=d ** -0.5, dtype=dt)
            self.K = inputs.project(Xh, Wk).view(N, H, dh).cuda()
            self.V = inputs.project(Xh, Wv).view(N, H, dh).cuda()
        else:
            self.K = draw((N, H, dh), "K")
            self.V = draw((N, H, dh), "V")
        self.loc_cap = wl.local + self.tq + self.steps
        self.locK = draw((B * self.loc_cap, H, dh), "locK")
        self.locV = draw((B * self.loc_cap, H, dh), "locV")
        self.Qd = draw((max(self.steps, 1), B, H, dh), "Qd")
        self.Od = torch.zeros_like(self.Qd)
        self.Qb = draw((max(B * self.tq, 1), H, dh), "Qb")
        self.Ob = torch.zeros_like(self.Qb)
        # log-sum-exp outputs (the parity tests ask for them; the timed runs pass NULL)
        self.lse_b = torch.full((max(B * self.tq, 1), H), float("nan"), device="cuda") if with_lse else None
        self.lse_d = torch.full((max(self.steps, 1), B, H), float("nan"), device="cuda") if with_lse else None
        self.qb_off = np.arange(B + 1, dtype=np.int32) * self.tq
        self.scores = torch.empty(N, dtype=torch.float32, device="cuda")
        self.idx = torch.empty(max(Kt, 1), dtype=torch.int32, device="cuda")
        self.cacheK = torch.zeros((max(Kt, 1), H, dh), dtype=dt, device="cuda")
        self.cacheV = torch.zeros_like(self.cacheK)
        self.cache_pos = torch.zeros(max(Kt, 1), dtype=torch.int32, device="cuda")
        self.cache_len = np.zeros(B, dtype=np.int32)
        self.ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
        self.q_off = np.arange(B + 1, dtype=np.int32)
        self.pos_base = np.zeros(B, dtype=np.int32)
        self.sm_scale = dh ** -0.5

    # -- the path --------------------------------------------------------------------------------
    def compress(self):
        """score, TopK select and gather into the empty nugget cache: dodo_compress (one launch where the batch allows)."""
        self.cache_len[:] = 0
        self.dodo.compress(self.X, self.w, 0.0, self.K, self.V, self.seq_off, self.nug_off, self.pos_base, 0, self.scores,
                           self.idx, self.cacheK, self.cacheV, self.cache_pos, self.cache_off, self.cache_len)

    def block_tables(self):
        """(loc_off, loc_len, loc_pos0, q_pos0) host tables of the query block."""
        B, L = self.wl.B, self.wl.local
        base = np.arange(B, dtype=np.int32) * self.loc_cap
        return base, np.full(B, L + self.tq, np.int32), self.n.copy(), self.n + L

    def query_block(self):
        """All tq query tokens of every sequence attend at once (causal inside the block)."""
        loc_off, loc_len, loc_pos0, q_pos0 = self.block_tables()
        self.dodo.attend(self.Qb, self.qb_off, q_pos0, self.sm_scale, self.cacheK, self.cacheV, self.cache_pos,
                         self.cache_off, self.cache_len, self.locK, self.locV, loc_off, loc_len, loc_pos0,
                         self.Ob, self.lse_b, self.ws)

    def window(self, s: int):
        """(loc_off, loc_len, loc_pos0, q_pos0) host tables of decode step s."""
        B, L = self.wl.B, self.wl.local
        base = np.arange(B, dtype=np.int32) * self.loc_cap
        q_pos0 = self.n + L + self.tq + s
        if self.sliding:
            return base + s + 1, np.full(B, L, np.int32), self.n + s + 1, q_pos0
        return base, np.full(B, L + self.tq + s + 1, np.int32), self.n.copy(), q_pos0

    def decode_step(self, s: int):
        loc_off, loc_len, loc_pos0, q_pos0 = self.window(s)
        self.dodo.attend(self.Qd[s], self.q_off, q_pos0, self.sm_scale, self.cacheK, self.cacheV, self.cache_pos,
                         self.cache_off, self.cache_len, self.locK, self.locV, loc_off, loc_len, loc_pos0,
                         self.Od[s], None if self.lse_d is None else self.lse_d[s], self.ws)

    # -- sizes -----------------------------------------------------------------------------------
    def bytes_score(self) -> int:
        e = self.X.element_size()
        return int(self.seq_off[-1]) * (self.wl.d * e + 4)

    def bytes_gather(self) -> int:
        row = self.wl.H * self.wl.dh * self.K.element_size()
        return int(self.nug_off[-1]) * (4 * row + 8)

    def bytes_decode_step(self, s: int) -> int:
        """Algorithmic bytes of one attend launch: K and V rows of every visible key, q in, o out."""
        row = self.wl.H * self.wl.dh * self.K.element_size()
        _, loc_len, _, _ = self.window(s)
        keys = int(self.k.sum()) + int(loc_len.sum())
        return 2 * keys * row + 2 * self.wl.B * row

    def flops_query_block(self) -> int:
        """4 * dh flop per (query, visible key, head): nuggets and local context in full, the block causally."""
        wl = self.wl
        keys = sum(self.tq * (int(k) + wl.local) + self.tq * (self.tq + 1) // 2 for k in self.k)
        return 4 * wl.dh * wl.H * keys

    def device_bytes(self) -> int:
        ts = [self.X, self.w, self.K, self.V, self.locK, self.locV, self.Qd, self.Od, self.Qb, self.Ob, self.scores, self.idx,
              self.cacheK, self.cacheV, self.cache_pos, self.ws]
        return sum(t.numel() * t.element_size() for t in ts)


class RaggedServing:
    """One layer of the ragged serving workload: sequences of very different context lengths are
    compressed once, then every sequence decodes one token per step; decoded tokens pile up
    uncompressed, and whenever a sequence's pile reaches 2*S tokens its oldest S are scored, the
    best ceil(S/r) of them are appended to its nugget cache, and they leave the local window.

    Layout: context X/K/V packed `[sum n_b, ...]`; decoded tokens `decX [B, steps, d]`,
    `decK/V [B, steps, H, dh]` (sequence-major, so a sequence's local window is a contiguous row
    range); the segment being compressed is copied into packed staging buffers `[B*S, ...]` first,
    because the library's score/gather calls take ragged-packed rows.  Decode token s of sequence b
    sits at position n_b + s.
    """

    def __init__(self, dodo, lengths, d, H, dh, r, steps, tag, dtype=torch.bfloat16, segment=64, gen_device="cuda",
                 with_lse: bool = False):
        self.dodo, self.r, self.steps, self.S = dodo, r, steps, segment
        self.B, self.d, self.H, self.dh = len(lengths), d, H, dh
        B = self.B
        self.n = np.asarray(lengths, dtype=np.int32)
        self.seq_off = inputs.offsets(self.n)
        self.k0 = np.asarray([dodo.num_nuggets(int(n), r) for n in self.n], dtype=np.int32)
        self.kS = dodo.num_nuggets(segment, r)
        self.appends = max(0, (steps - segment) // segment)
        self.cache_off = inputs.offsets(self.k0 + self.appends * self.kS)
        self.nug_off0 = inputs.offsets(self.k0)
        N, cap = int(self.seq_off[-1]), int(self.cache_off[-1])

        def draw(shape, name, std=1.0):
            return inputs.randn(shape, *tag, name, std=std, dtype=dtype, device=gen_device).cuda()

        self.X, self.w = draw((N, d), "X"), draw((d,), "w", std=d ** -0.5)
        self.K, self.V = draw((N, H, dh), "K"), draw((N, H, dh), "V")
        self.decX = draw((B, steps, d), "decX")
        self.decK, self.decV = draw((B, steps, H, dh), "decK"), draw((B, steps, H, dh), "decV")
        self.Qd = draw((steps, B, H, dh), "Qd")
        self.Od = torch.zeros_like(self.Qd)
        self.lse_d = torch.full((steps, B, H), float("nan"), device="cuda") if with_lse else None
        self.scores = torch.empty(max(N, B * segment), dtype=torch.float32, device="cuda")
        self.idx = torch.empty(max(int(self.nug_off0[-1]), B * self.kS), dtype=torch.int32, device="cuda")
        self.cacheK = torch.zeros((cap, H, dh), dtype=dtype, device="cuda")
        self.cacheV = torch.zeros_like(self.cacheK)
        self.cache_pos = torch.zeros(cap, dtype=torch.int32, device="cuda")
        self.cache_len = np.zeros(B, dtype=np.int32)
        self.stageX = torch.empty((B * segment, d), dtype=dtype, device="cuda")
        self.stageK = torch.empty((B * segment, H, dh), dtype=dtype, device="cuda")
        self.stageV = torch.empty_like(self.stageK)
        self.seg_off = np.arange(B + 1, dtype=np.int32) * segment
        self.seg_nug_off = np.arange(B + 1, dtype=np.int32) * self.kS
        self.ws = torch.empty(dodo.attend_workspace_bytes(dh), dtype=torch.uint8, device="cuda")
        self.q_off = np.arange(B + 1, dtype=np.int32)
        self.win0 = 0            # first decoded token still in the local window (same for all sequences)
        self.sm_scale = dh ** -0.5

    def compress_context(self):
        self.cache_len[:] = 0
        self.win0 = 0
        self.dodo.compress(self.X, self.w, 0.0, self.K, self.V, self.seq_off, self.nug_off0, np.zeros(self.B, np.int32), 0,
                           self.scores, self.idx, self.cacheK, self.cacheV, self.cache_pos, self.cache_off, self.cache_len)

    def rewind(self):
        """Host tables back to the state right after compress_context() (nothing is launched): the decode loop
        can then be recorded or run again; it rewrites the same appended rows."""
        self.cache_len[:] = self.k0
        self.win0 = 0

    def window(self, s: int):
        """(loc_off, loc_len, loc_pos0, q_pos0) of decode step s over the flat [B*steps] decoded rows."""
        base = np.arange(self.B, dtype=np.int32) * self.steps
        return base + self.win0, np.full(self.B, s + 1 - self.win0, np.int32), self.n + self.win0, self.n + s

    def decode_step(self, s: int) -> bool:
        """Attend for token s of every sequence; returns True when this step ended with an append."""
        loc_off, loc_len, loc_pos0, q_pos0 = self.window(s)
        B, st = self.B, self.steps
        self.dodo.attend(self.Qd[s], self.q_off, q_pos0, self.sm_scale, self.cacheK, self.cacheV, self.cache_pos,
                         self.cache_off, self.cache_len, self.decK.view(B * st, self.H, self.dh),
                         self.decV.view(B * st, self.H, self.dh), loc_off, loc_len, loc_pos0, self.Od[s],
                         None if self.lse_d is None else self.lse_d[s], self.ws)
        if s + 1 - self.win0 < 2 * self.S:
            return False
        self.append_segment()
        return True

    def append_segment(self):
        """Compress the oldest S decoded tokens of every sequence into its nugget cache."""
        S, w0, B = self.S, self.win0, self.B
        self.stageX.view(B, S, self.d).copy_(self.decX[:, w0:w0 + S])
        self.stageK.view(B, S, self.H, self.dh).copy_(self.decK[:, w0:w0 + S])
        self.stageV.view(B, S, self.H, self.dh).copy_(self.decV[:, w0:w0 + S])
        self.dodo.compress(self.stageX, self.w, 0.0, self.stageK, self.stageV, self.seg_off, self.seg_nug_off, self.n + w0, 0,
                           self.scores, self.idx, self.cacheK, self.cacheV, self.cache_pos, self.cache_off, self.cache_len)
        self.win0 += S

    def keys_per_step(self, s: int) -> int:
        return int(self.cache_len.sum()) + self.B * (s + 1 - self.win0)
