"""Policy in the loop: the GRU policy of gru_policy.h produces, on the same
stream, the actions that drive the batched env step of pong.h; K agent steps
are captured as one CUDA graph.

This is the setting of the paper's "GRU rollout (~2M-parameter policy)" rows
(Table "PufferLib comparisons") and of its observation that with a fast
environment the step time is dominated by the model (Sec. 4, time breakdown).
Per agent step, five kernels of this package and nothing else:

    x          <- gru_policy_encode(obs, done, h)      also clears h where the last step ended an episode
    h', logits <- gru_policy_cell_head(x, h)           tensor cores; the head's partial sums are formed in
                                                       the cell's epilogue, a small kernel adds them up
    actions    <- pong_sample_actions(logits, words[i])
    obs, reward, done <- pong_step(actions)

The uniform numbers of the draws are generated before each replay with
pong_fill_words (outside the graph), so a replayed graph draws fresh,
reproducible numbers; the handle's step counter is put right after capture and
after every replay.  The loop's running result is the env's episode statistics.
"""
from __future__ import annotations

from . import gru_policy, pong


class PolicyLoop:
    """Owns the buffers of the loop and, after capture(), its CUDA graph."""

    def __init__(self, env: "pong.PongEnv", policy: "gru_policy.GruPolicy", steps_per_graph: int = 32):
        import torch
        if env.obs_mode != pong.OBS_VECTOR or env.frameskip != 1:
            raise ValueError("the captured loop needs vector observations and frameskip 1")
        if policy.obs_dim != 6 or policy.n_actions != 3:
            raise ValueError("the Pong env has 6 observations and 3 actions")
        if steps_per_graph < 2 or steps_per_graph % 2:
            raise ValueError("steps_per_graph must be even: the hidden state alternates between two buffers")
        self.torch, self.env, self.policy, self.K = torch, env, policy, int(steps_per_graph)
        n, dev, H = env.n, env.device, policy.hidden
        self.obs = torch.empty((n, 6), dtype=torch.float32, device=dev)
        self.reward = torch.empty((n,), dtype=torch.float32, device=dev)
        self.done = torch.zeros((n,), dtype=torch.uint8, device=dev)
        self.x = torch.empty((n, H), dtype=torch.bfloat16, device=dev)
        self.h = [torch.zeros((n, H), dtype=torch.bfloat16, device=dev) for _ in range(2)]
        self.cur = 0                                     # which of the two holds the current hidden state
        self.logits = torch.zeros((n, 3), dtype=torch.float32, device=dev)
        self.scratch = policy.workspace(n)                # the head's partial sums, written by the cell kernel
        self.actions = torch.empty((n,), dtype=torch.uint8, device=dev)
        self.words = torch.empty((self.K, n), dtype=torch.int32, device=dev)
        self.graph = None
        self.with_env = True
        env._stream()
        self.obs.copy_(env.reset())

    @property
    def hidden(self):
        return self.h[self.cur]

    def _step(self, i: int, with_env: bool = True, with_policy: bool = True):
        n = self.env.n
        if with_policy:
            p = self.policy.h
            gru_policy.gru_policy_encode(p, self.obs, self.done, self.h[self.cur], self.x, n)
            gru_policy.gru_policy_cell_head(p, self.x, self.h[self.cur], self.h[self.cur ^ 1], self.logits,
                                            self.scratch, n)
            self.cur ^= 1
        if with_env:
            pong.pong_sample_actions(self.env.h, self.logits, self.words[i], self.actions)
            pong.pong_step(self.env.h, self.actions, self.obs, self.reward, self.done)

    def _streams(self):
        self.env._stream()
        self.policy._stream()

    def run_eager(self, steps: int):
        """`steps` agent steps without a graph (the host launches every kernel)."""
        self._streams()
        done = 0
        while done < steps:
            k = min(self.K, steps - done)
            pong.pong_fill_words(self.env.h, k, self.words)
            for i in range(k):
                self._step(i)
            done += k

    def capture(self, with_env: bool = True, with_policy: bool = True):
        """Capture K agent steps.  with_env=False captures the policy alone (no
        sampling and no env step), with_policy=False the env-side kernels alone
        (sampling from the current logits + env step): the two parts of the step,
        to report the env's share."""
        t = self.torch
        t0 = self.env.t
        # every kernel runs once on a scratch loop first, so that nothing is loaded
        # for the first time while the stream is capturing
        side = t.cuda.Stream(device=self.env.device)
        side.wait_stream(t.cuda.current_stream(self.env.device))
        with t.cuda.stream(side):
            scratch = PolicyLoop(pong.PongEnv(64, 0, device=str(self.env.device)), self.policy, 2)
            scratch.run_eager(2)
            self.policy.status()
            scratch.env.close()
        t.cuda.current_stream(self.env.device).wait_stream(side)
        self.graph = t.cuda.CUDAGraph()
        cur = self.cur
        with t.cuda.graph(self.graph):
            self._streams()
            for i in range(self.K):
                self._step(i, with_env, with_policy)
        assert self.cur == cur or not with_policy
        self._streams()
        self.env.t = t0                       # capturing ran the host-side counting, not the kernels
        self.with_env = with_env

    def replay(self):
        """K more agent steps from the captured graph.  Enqueues only: the results are valid
        once sync_and_check() (or policy.status()) has returned without raising."""
        if self.with_env:
            pong.pong_fill_words(self.env.h, self.K, self.words)
        self.graph.replay()
        if self.with_env:
            self.env.t = self.env.t + self.K

    def sync_and_check(self):
        """Synchronises the policy's stream and raises GruPolicyError (ETIMEOUT) if a cell
        kernel since the last check gave up a bounded wait: its h' and logits, and everything
        the env did with them, are then invalid.  The error word belongs to the policy handle,
        so loops that share a policy share it; whoever checks first sees (and clears) it."""
        self._streams()
        self.policy.status()


class PipelinedPolicyLoop:
    """The same loop over `parts` disjoint slices of the envs, each slice a
    PolicyLoop of its own on its own stream, all captured into one CUDA graph.

    The slices are independent (envs are), so the graph has `parts` parallel
    chains and the device overlaps one slice's small memory-bound kernels
    (encoder, head, sampling, env step) with another slice's tensor-core cell.
    Env ids are global (`env_id_base` + slice offset): the union of the slices'
    trajectories is the trajectory of one loop over all envs."""

    def __init__(self, n_envs: int, seed: int, policy: "gru_policy.GruPolicy", steps_per_graph: int = 32,
                 parts: int = 2, env_id_base: int = 0, device=None):
        import torch
        if parts < 1 or n_envs % parts:
            raise ValueError("n_envs must be a multiple of parts")
        self.torch, self.policy, self.K, self.n = torch, policy, int(steps_per_graph), int(n_envs)
        per = n_envs // parts
        dev = str(device) if device is not None else str(policy.device)
        self.parts = [PolicyLoop(pong.PongEnv(per, seed, env_id_base=env_id_base + i * per, device=dev),
                                 policy, steps_per_graph) for i in range(parts)]
        self.device = self.parts[0].env.device
        self.streams = [torch.cuda.Stream(device=self.device) for _ in self.parts]
        self.graph = None
        self.with_env = True

    def run_eager(self, steps: int):
        for part in self.parts:
            part.run_eager(steps)

    def capture(self, with_env: bool = True, with_policy: bool = True):
        t = self.torch
        t0 = [part.env.t for part in self.parts]
        side = t.cuda.Stream(device=self.device)
        side.wait_stream(t.cuda.current_stream(self.device))
        with t.cuda.stream(side):
            scratch = PolicyLoop(pong.PongEnv(64, 0, device=str(self.device)), self.policy, 2)
            scratch.run_eager(2)
            self.policy.status()
            scratch.env.close()
        t.cuda.current_stream(self.device).wait_stream(side)
        self.graph = t.cuda.CUDAGraph()
        with t.cuda.graph(self.graph):
            main = t.cuda.current_stream(self.device)
            for part, stream in zip(self.parts, self.streams):
                stream.wait_stream(main)
            # issue the chains step by step in turn, so that the capture order (which the
            # device's scheduler tends to follow) already interleaves them
            for i in range(self.K):
                for part, stream in zip(self.parts, self.streams):
                    with t.cuda.stream(stream):
                        part._streams()
                        part._step(i, with_env, with_policy)
            for stream in self.streams:
                main.wait_stream(stream)
        for part, start in zip(self.parts, t0):
            part._streams()
            part.env.t = start
        self.with_env = with_env

    def replay(self):
        """K more agent steps of every slice.  Enqueues only: see sync_and_check()."""
        if self.with_env:
            for part in self.parts:
                part._streams()
                pong.pong_fill_words(part.env.h, self.K, part.words)
        self.graph.replay()
        if self.with_env:
            for part in self.parts:
                part.env.t = part.env.t + self.K

    def sync_and_check(self):
        """Synchronises the device and raises if any slice's cell kernel gave up a wait (one
        error word for all slices: it says that some result since the last check is invalid)."""
        self.torch.cuda.synchronize(self.device)
        self.parts[0]._streams()
        self.policy.status()

    def episode_stats(self):
        totals = [0, 0, 0]
        for part in self.parts:
            part._streams()
            for i, v in enumerate(part.env.episode_stats()):
                totals[i] += int(v)
        return tuple(totals)

    @property
    def launches(self) -> int:
        return sum(part.env.launches for part in self.parts)
