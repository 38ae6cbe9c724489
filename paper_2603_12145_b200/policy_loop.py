"""Policy in the loop: a small GRU policy on the same stream produces the actions
that drive the batched env step, captured as a CUDA graph.

This is the setting of the paper's "GRU rollout (~2M-parameter policy)" rows
(Table "PufferLib comparisons") and of its observation that with a fast
environment the step time is dominated by the model (Sec. 4, time breakdown).
Per agent step, all on one stream and without touching the host:

    hidden  <- GRU(obs, hidden)                      torch (cuBLAS GEMMs: library)
    logits  <- head(hidden)                          torch
    actions <- pong_sample_actions(logits, words[i]) this library's kernel
    obs, reward, done <- pong_step(actions)          this library's kernel
    hidden  <- hidden * (1 - done)                   torch

The policy's matrix products are library calls and are not part of what this
package implements; the env-side kernels are.  The uniform numbers of the draws
are generated before each replay with pong_fill_words (outside the graph), so a
replayed graph draws fresh, reproducible numbers; the handle's step counter is
put right after capture and after every replay.
"""
from __future__ import annotations

from typing import Optional

from . import pong


def make_policy(hidden: int = 576, seed: int = 0, dtype=None):
    """Linear(6, H) -> GRUCell(H, H) -> Linear(H, 3); H = 576 gives about 2.0 M
    parameters.  Weights are drawn from a seeded generator on the CPU, so the same
    seed gives the same policy everywhere."""
    import torch

    class GruPolicy(torch.nn.Module):
        def __init__(self):
            super().__init__()
            self.encoder = torch.nn.Linear(6, hidden)
            self.cell = torch.nn.GRUCell(hidden, hidden)
            self.head = torch.nn.Linear(hidden, 3)

        def forward(self, obs, h):
            x = torch.relu(self.encoder(obs.to(self.encoder.weight.dtype)))
            h = self.cell(x, h)
            return self.head(h).float(), h

    gen = torch.Generator().manual_seed(seed)
    policy = GruPolicy()
    with torch.no_grad():
        for p in policy.parameters():
            p.copy_(torch.empty(p.shape).uniform_(-0.05, 0.05, generator=gen))
    policy = policy.cuda().eval()
    if dtype is not None:
        policy = policy.to(dtype)
    return policy


class PolicyLoop:
    """Owns the buffers of the loop and, after capture(), its CUDA graph."""

    def __init__(self, env: "pong.PongEnv", policy, steps_per_graph: int = 32):
        import torch
        if env.obs_mode != pong.OBS_VECTOR or env.frameskip != 1:
            raise ValueError("the captured loop needs vector observations and frameskip 1")
        self.torch, self.env, self.policy, self.K = torch, env, policy, int(steps_per_graph)
        n, dev = env.n, env.device
        hidden = policy.cell.hidden_size
        wdtype = policy.cell.weight_hh.dtype
        self.obs = torch.empty((n, 6), dtype=torch.float32, device=dev)
        self.reward = torch.empty((n,), dtype=torch.float32, device=dev)
        self.done = torch.empty((n,), dtype=torch.uint8, device=dev)
        self.hidden = torch.zeros((n, hidden), dtype=wdtype, device=dev)
        self.logits = torch.zeros((n, 3), dtype=torch.float32, device=dev)
        self.actions = torch.empty((n,), dtype=torch.uint8, device=dev)
        self.words = torch.empty((self.K, n), dtype=torch.int32, device=dev)
        self.reward_sum = torch.zeros((), dtype=torch.float64, device=dev)
        self.graph = None
        env._stream()
        self.obs.copy_(env.reset())

    def _step(self, i: int, with_env: bool = True, with_policy: bool = True):
        t = self.torch
        if with_policy:
            with t.no_grad():
                logits, h = self.policy(self.obs, self.hidden)
                self.logits.copy_(logits)
                self.hidden.copy_(h)
        if with_env:
            pong.pong_sample_actions(self.env.h, self.logits, self.words[i], self.actions)
            pong.pong_step(self.env.h, self.actions, self.obs, self.reward, self.done)
        if with_env and with_policy:
            with t.no_grad():
                self.hidden.mul_((1 - self.done).to(self.hidden.dtype).unsqueeze(1))
                self.reward_sum.add_(self.reward.sum(dtype=t.float64))

    def run_eager(self, steps: int):
        """`steps` agent steps without a graph (host launches every kernel)."""
        self.env._stream()
        done = 0
        while done < steps:
            k = min(self.K, steps - done)
            pong.pong_fill_words(self.env.h, k, self.words)
            for i in range(k):
                self._step(i)
            done += k

    def capture(self, with_env: bool = True, with_policy: bool = True):
        """Capture K agent steps.  with_env=False captures the policy alone (same
        GEMMs, no sampling and no env step), with_policy=False the env-side kernels
        alone (sampling from the current logits + env step): the two parts of the
        step, to report the env's share."""

        t = self.torch
        t0 = self.env.t
        side = t.cuda.Stream()
        side.wait_stream(t.cuda.current_stream())
        with t.cuda.stream(side):            # warm-up outside capture (cuBLAS workspaces etc.)
            self.env._stream()
            saved = (self.obs.clone(), self.hidden.clone(), self.reward_sum.clone())
            state, _ = self.env.get_state()
            pong.pong_fill_words(self.env.h, self.K, self.words)
            for i in range(2):
                self._step(i, with_env, with_policy)
            self.env.set_state(state, t0)
            self.obs.copy_(saved[0]); self.hidden.copy_(saved[1]); self.reward_sum.copy_(saved[2])
        t.cuda.current_stream().wait_stream(side)
        self.graph = t.cuda.CUDAGraph()
        with t.cuda.graph(self.graph):
            self.env._stream()
            for i in range(self.K):
                self._step(i, with_env, with_policy)
        self.env._stream()
        self.env.t = t0                       # capturing ran the host-side counting, not the kernels
        self.with_env = with_env

    def replay(self):
        """K more agent steps from the captured graph."""
        if self.with_env:
            pong.pong_fill_words(self.env.h, self.K, self.words)
        self.graph.replay()
        if self.with_env:
            self.env.t = self.env.t + self.K
