"""One pruned-GRPO batch step on the device: buffers + the four library calls in order.

This is plumbing around :mod:`.binding`: it allocates device memory with torch, copies the small
per-batch inputs in, issues the library calls on the current CUDA stream and copies results back.
All arithmetic happens inside libdppo.
"""
import torch

from . import binding as B
from . import dp


class DppoStep:
    """Buffers for a batch of P prompts x G completions and a loss sweep over at most T_max tokens.

    prune_pack():  rewards -> advantages -> candidate sets, masks, gamma, w_seq, H_next -> packing of the
                   retained completions (unit = prompt + response tokens) into rows of L_row, with
                   cu_seqlens over the response tokens in packed order.
    loss():        fused sweep over logits [T, V] of the retained response tokens in packed order.
    """

    def __init__(self, P, G, L_row, N_win, r_q, r_o, V, dtype, T_max, eps_lo=0.2, eps_hi=0.2, beta=0.04,
                 temperature=1.0, mode=0, reverse=0, policy=0, std_ddof=0, std_eps=1e-6, device="cuda", group=None):
        if not torch.cuda.is_available():
            raise RuntimeError("DppoStep needs a CUDA device: libdppo has no CPU path")
        self.P, self.G, self.n = P, G, P * G
        self.V, self.T_max = V, T_max
        self.dtype = dtype
        self.std_ddof, self.std_eps = std_ddof, std_eps
        dev = torch.device(device)
        self.device = dev
        self.group = group                       # torch.distributed process group of the data-parallel ranks (or None)
        self.H_table = None                      # dataset-wide history scores, owned by run_epochs
        n = self.n
        f32 = dict(dtype=torch.float32, device=dev)
        i32 = dict(dtype=torch.int32, device=dev)
        u8 = dict(dtype=torch.uint8, device=dev)
        self.rewards = torch.zeros(n, **f32)
        self.H_prev = torch.zeros(P, **f32)
        self.has_history = False
        self.unit_len = torch.zeros(n, **i32)
        self.loss_len = torch.zeros(n, **i32)
        self.adv = torch.zeros(n, **f32)
        self.mean_abs_adv = torch.zeros(P, **f32)
        self.cand_q = torch.zeros(P, **u8); self.cand_o = torch.zeros(n, **u8)
        self.keep_q = torch.zeros(P, **u8); self.keep_o = torch.zeros(n, **u8)
        self.n_keep_q = torch.zeros(1, **i32); self.n_keep_o = torch.zeros(P, **i32)
        self.gamma_q = torch.zeros(P, **f32); self.gamma_o = torch.zeros(n, **f32)
        self.w_seq = torch.zeros(n, **f32); self.H_next = torch.zeros(P, **f32)
        self.order = torch.zeros(n, **i32); self.row_of = torch.zeros(n, **i32)
        self.off_in_row = torch.zeros(n, **i32); self.row_fill = torch.zeros(n, **i32)
        self.cu_seqlens = torch.zeros(n + 1, **i32); self.counts = torch.zeros(4, **i32)
        self.status = torch.zeros(1, **i32)
        self.loss_out = torch.zeros(5, **f32)
        self.logp_out = torch.zeros(max(T_max, 1), **f32); self.lse_out = torch.zeros(max(T_max, 1), **f32)

        self.prune_params = B.PruneParams(P, G, r_q, r_o, mode, reverse, 0, 0)
        self.pack_params = B.PackParams(n, L_row, N_win, policy)
        self.loss_params = B.LossParams(T_max, V, B.BF16 if dtype == "bf16" else B.F32, V, n, 0,
                                        eps_lo, eps_hi, beta, temperature)
        self.pack_ws_bytes = B.pack_workspace_bytes(self.pack_params)
        self.pack_ws = torch.zeros(max(self.pack_ws_bytes, 16), dtype=torch.uint8, device=dev)
        self.loss_ws_bytes = B.grpo_loss_workspace_bytes(self.loss_params)
        self.loss_ws = torch.zeros(max(self.loss_ws_bytes, 16), dtype=torch.uint8, device=dev)

    # -- inputs ------------------------------------------------------------------------------------
    def set_batch(self, rewards, unit_len, loss_len, H_prev=None):
        """Copy the per-batch host inputs (numpy / torch) to the device."""
        self.rewards.copy_(torch.as_tensor(rewards, dtype=torch.float32).reshape(-1), non_blocking=True)
        self.unit_len.copy_(torch.as_tensor(unit_len, dtype=torch.int32).reshape(-1), non_blocking=True)
        self.loss_len.copy_(torch.as_tensor(loss_len, dtype=torch.int32).reshape(-1), non_blocking=True)
        self.has_history = H_prev is not None
        if self.has_history:
            self.H_prev.copy_(torch.as_tensor(H_prev, dtype=torch.float32).reshape(-1), non_blocking=True)

    # -- library calls -----------------------------------------------------------------------------
    def advantages(self, rewards=None, adv=None, mean_abs_adv=None):
        B.group_advantages(self.rewards if rewards is None else rewards, self.P, self.G,
                           self.adv if adv is None else adv,
                           self.mean_abs_adv if mean_abs_adv is None else mean_abs_adv,
                           self.std_ddof, self.std_eps, self.status)

    def prune(self, seed, step, u_q=None, u_o=None):
        self.prune_params.seed, self.prune_params.step = seed, step
        B.prune_and_rescale(self.prune_params, self.adv, self.mean_abs_adv,
                            self.H_prev if self.has_history else None, u_q, u_o,
                            self.cand_q, self.cand_o, self.keep_q, self.keep_o, self.n_keep_q, self.n_keep_o,
                            self.gamma_q, self.gamma_o, self.w_seq, self.H_next, self.status)

    def pack(self):
        B.pack_prompts(self.pack_params, self.unit_len, self.keep_o, self.loss_len, self.order, self.row_of,
                       self.off_in_row, self.row_fill, self.cu_seqlens, self.counts, self.pack_ws,
                       self.pack_ws_bytes, self.status)

    def prune_pack(self, seed=0, step=0, u_q=None, u_o=None):
        self.advantages()
        self.prune(seed, step, u_q, u_o)
        self.pack()

    def loss(self, logits, target, logp_old, logp_ref, dlogits=None, row_stride=None):
        """Loss sweep over the retained tokens; the true token count is read on the device from the
        packer's counts.  dlogits may be `logits` itself (in place) or None (forward only)."""
        self.loss_params.row_stride = self.V if row_stride is None else row_stride
        B.grpo_loss_fwd_bwd(self.loss_params, logits, target, logp_old, logp_ref, self.cu_seqlens,
                            self.counts[3:4], self.adv, self.w_seq, self.order, dlogits, self.logp_out,
                            self.lse_out, self.loss_out, self.loss_ws, self.loss_ws_bytes, self.status)

    def step_from_host(self, batch_host, token_host, dev_tokens, seed=0, step=0, dlogits=None):
        """The whole path from HOST buffers: copies the batch inputs and the token inputs (logits, targets,
        old / reference log-probs; pinned host tensors) to the device, runs advantages -> prune -> pack ->
        loss sweep, and returns the five loss scalars on the host (this synchronises).

        batch_host: dict with pinned tensors rewards, unit_len, loss_len and optionally H_prev.
        token_host / dev_tokens: dicts with logits, target, logp_old, logp_ref (host source, device
        destination).  A host tensor with fewer rows than its destination is treated as a window that is
        copied repeatedly (same bytes over the bus, for hosts that cannot pin the whole input).  Returns (loss_out as a host tensor, bytes copied host->device, bytes device->host).
        """
        h2d = 0
        for name in ("rewards", "unit_len", "loss_len"):
            getattr(self, name).copy_(batch_host[name], non_blocking=True)
            h2d += batch_host[name].numel() * batch_host[name].element_size()
        self.has_history = batch_host.get("H_prev") is not None
        if self.has_history:
            self.H_prev.copy_(batch_host["H_prev"], non_blocking=True)
            h2d += batch_host["H_prev"].numel() * 4
        for name in ("logits", "target", "logp_old", "logp_ref"):
            src, dst = token_host[name], dev_tokens[name]
            if src.shape[0] >= dst.shape[0]:
                dst.copy_(src[:dst.shape[0]], non_blocking=True)
            else:
                # the pinned host buffer is a window of `src.shape[0]` rows (host memory is short): the
                # same number of bytes crosses the bus, window by window
                for a in range(0, dst.shape[0], src.shape[0]):
                    b = min(dst.shape[0], a + src.shape[0])
                    dst[a:b].copy_(src[:b - a], non_blocking=True)
            h2d += dst.numel() * dst.element_size()
        self.prune_pack(seed, step)
        self.loss(dev_tokens["logits"], dev_tokens["target"], dev_tokens["logp_old"], dev_tokens["logp_ref"], dlogits)
        out = self.loss_out.cpu()                         # device -> host read of the result; synchronises
        return out, h2d, out.numel() * 4

    # -- several ranks ---------------------------------------------------------------------------
    def shard(self, world, rank):
        """This rank's contiguous range of the packed rows of the last prune_pack (reads the packer's
        outputs: synchronises).  See dp.shard_rows."""
        n_units = int(self.counts[0].item())
        order = self.order[:n_units].long()
        return dp.shard_rows(self.row_of[order].cpu().tolist(), self.cu_seqlens.cpu().tolist(), n_units, world, rank)

    def loss_shard(self, shard, logits, target, logp_old, logp_ref, dlogits=None, row_stride=None):
        """Loss sweep over one rank's share of the packed rows: `logits` (and the other per-token inputs) hold the
        tokens [tok_lo, tok_hi) of the batch, in packed order.  The sequence weights are those of the WHOLE batch,
        so the five scalars of all ranks add up to the batch's (all_reduce_loss)."""
        lo, hi = shard["seq_lo"], shard["seq_hi"]
        T_r = shard["tok_hi"] - shard["tok_lo"]
        prm = B.LossParams.from_buffer_copy(self.loss_params)
        prm.T_max, prm.S_max = T_r, max(hi - lo, 1)
        prm.row_stride = self.V if row_stride is None else row_stride
        cu_local = (self.cu_seqlens[lo:hi + 1] - shard["tok_lo"]).contiguous() if hi > lo else self.cu_seqlens[:2] * 0
        seg_map = self.order[lo:max(hi, lo + 1)].contiguous()
        B.grpo_loss_fwd_bwd(prm, logits, target, logp_old, logp_ref, cu_local, None, self.adv, self.w_seq, seg_map,
                            dlogits, self.logp_out, self.lse_out, self.loss_out, self.loss_ws, self.loss_ws_bytes,
                            self.status)

    def all_reduce_loss(self, average=False):
        """Combines loss_out over the ranks of `group` (a no-op for a single process); see dp.all_reduce_loss."""
        return dp.all_reduce_loss(self.loss_out, self.group, average)

    # -- several epochs ----------------------------------------------------------------------------
    def run_epochs(self, n_prompts, batches_by_epoch, rewards_fn, seed, lengths_fn=None, on_batch=None):
        """Algorithm 1's outer loops around the small steps, with the dataset-wide history table of Eq. 16.

        The table H (one score per dataset prompt, zero at the start) lives on the device and is owned by this
        object (self.H_table).  For batch b of epoch t (a list of P dataset prompt ids): gather the prompts'
        scores -> advantages -> candidate sets, masks and weights (no prompt pruning in the first epoch; the
        generator's step word is t * 1,000,000 + b) -> scatter the updated scores back (retained prompts get their
        fresh mean |A|, pruned ones keep the old score) -> pack the retained completions.  Every step is a library
        call on the current stream; nothing is read back unless `on_batch` does.

        rewards_fn(t, ids) -> float32 [P, G] rewards of those prompts in epoch t (host array)
        lengths_fn(t, ids) -> (unit_len, loss_len) int32 [P*G] each, or None to skip the packing step
        on_batch(t, b, self)  called after each batch with the results in this object's buffers
        Returns self.H_table.
        """
        self.H_table = torch.zeros(n_prompts, dtype=torch.float32, device=self.device)
        ids_dev = torch.zeros(self.P, dtype=torch.int32, device=self.device)
        for t, batches in enumerate(batches_by_epoch):
            for b, ids in enumerate(batches):
                if len(ids) != self.P:
                    raise ValueError("a batch must hold P = %d prompt ids, got %d" % (self.P, len(ids)))
                ids_dev.copy_(torch.as_tensor(ids, dtype=torch.int32), non_blocking=False)
                self.rewards.copy_(torch.as_tensor(rewards_fn(t, ids), dtype=torch.float32).reshape(-1))
                if lengths_fn is not None:
                    unit_len, loss_len = lengths_fn(t, ids)
                    self.unit_len.copy_(torch.as_tensor(unit_len, dtype=torch.int32).reshape(-1))
                    self.loss_len.copy_(torch.as_tensor(loss_len, dtype=torch.int32).reshape(-1))
                B.history_gather(self.H_table, n_prompts, ids_dev, self.P, self.H_prev, self.status)
                self.has_history = t > 0
                self.advantages()
                self.prune(seed, t * 1000000 + b)
                B.history_scatter(self.H_table, n_prompts, ids_dev, self.P, self.H_next, self.status)
                if lengths_fn is not None:
                    self.pack()
                if on_batch is not None:
                    on_batch(t, b, self)
        return self.H_table

    # -- results -----------------------------------------------------------------------------------
    def n_tokens(self):
        """Retained loss tokens T of the last prune_pack (synchronises)."""
        return int(self.counts[3].item())

    def prune_results(self):
        names = ["adv", "mean_abs_adv", "cand_q", "cand_o", "keep_q", "keep_o", "n_keep_q", "n_keep_o",
                 "gamma_q", "gamma_o", "w_seq", "H_next"]
        return {k: getattr(self, k).cpu().numpy() for k in names}

    def pack_results(self):
        names = ["order", "row_of", "off_in_row", "row_fill", "cu_seqlens", "counts", "status"]
        return {k: getattr(self, k).cpu().numpy() for k in names}
