"""Vectorised step() interface over the C ABI (paper Appendix A.1): one call advances N
environments x M agents and returns N x M observations and N termination flags; finished
environments are reset automatically, so the last frame of an episode is never rendered.

Scenario logic, rewards and object physics are outside this library: an "episode" here is a
fixed number of steps, after which the environment gets a freshly generated world.  The
time-left bar of Appendix A.2 is drawn through the GUI overlay.  Observations are zero-copy CUDA
tensors owned by this object (Section 3.2: frames exposed directly as GPU-side tensors).

Built for thousands of environments: episode clocks, the time-left rectangles and the agent state
live on the GPU; per step the host only learns which environments finished (one small read) and
uploads their new worlds with one scattered upload.  Episode lengths are fixed, so the worlds that
the next few steps will need are known in advance and are generated together, a window at a time."""
from __future__ import annotations

import torch

from . import binding, scenes

BAR_RGB = (250, 240, 30)
BAR_ROWS = 2
_GEN_CHUNK = 512            # environments generated per scene-generator call
_LOOKAHEAD = 8              # steps whose resets are generated together


def time_bar_rects(steps_left, episode_len, width, agents):
    """int32 [E*agents][1][4] overlay records: a bar of BAR_ROWS rows whose length is the share of
    the episode that is left, rounded down to whole pixels.  Runs on the device of its inputs."""
    steps_left = torch.as_tensor(steps_left, dtype=torch.int64)
    episode_len = torch.as_tensor(episode_len, dtype=torch.int64).to(steps_left.device)
    x1 = (width * steps_left) // episode_len.clamp(min=1)
    x1 = x1.clamp(0, width).repeat_interleave(agents)
    n = x1.numel()
    rec = torch.zeros(n, 1, 4, dtype=torch.int32, device=steps_left.device)
    rec[:, 0, 1] = x1.to(torch.int32) | (BAR_ROWS << 16)   # x1 (low half), y1 (high half); x0 = y0 = 0
    rec[:, 0, 2] = BAR_RGB[0] | (BAR_RGB[1] << 8) | (BAR_RGB[2] << 16)
    return rec


class VecRenderEnv:
    def __init__(self, cfg: scenes.SceneConfig, episode_len, device: int = 0, time_bar: bool = True, phase=None):
        """episode_len: steps per episode (scalar or one per env).  phase: optional initial value of each
        env's step clock (so that episodes end at different times from the start)."""
        self.cfg, self.device = cfg, torch.device("cuda", device)
        E = cfg.num_envs
        self.episode_len = torch.as_tensor(episode_len, dtype=torch.int64).expand(E).clone().to(self.device)
        self.time_bar = time_bar
        self.batch = binding.Batch(binding.desc_from_config(cfg, device, max_overlay_rects=1 if time_bar else 0))
        self.cams = torch.zeros(cfg.num_obs, 6, dtype=torch.int32, device=self.device)
        self.rgb, self.depth = self.batch.alloc_outputs()
        self.t = torch.zeros(E, dtype=torch.int64, device=self.device)
        if phase is not None:
            self.t = torch.as_tensor(phase, dtype=torch.int64).expand(E).clone().to(self.device)
        self.episode = torch.zeros(E, dtype=torch.int64, device=self.device)
        self._bar_count = torch.ones(cfg.num_obs, dtype=torch.int32, device=self.device)
        self._started = False
        self._step = 0                      # steps taken so far
        self._ahead = {}                    # step number -> (env list, their generated scenes) for coming resets

    def _generate(self, envs, episodes):
        """Scenes (a list of chunks) for the env indices `envs` in the given episodes: env e in its k-th
        episode uses the seeded scene id e + k * num_envs."""
        out = []
        for c0 in range(0, len(envs), _GEN_CHUNK):
            chunk = envs[c0:c0 + _GEN_CHUNK]
            ids = torch.tensor([e + k * self.cfg.num_envs for e, k in zip(chunk, episodes[c0:c0 + _GEN_CHUNK])],
                               dtype=torch.int64)
            out.append((chunk, scenes.make_scene(self.cfg, device=self.device, env_ids=ids)))
        return out

    def _install(self, chunks, pick=None):
        """Upload generated scenes; `pick` (env list, position range) takes a slice of a single chunk."""
        A = self.cfg.agents
        for chunk, sc in chunks:
            lo, hi = (0, len(chunk)) if pick is None else pick
            envs = chunk[lo:hi]
            if not envs:
                continue
            boxes = count = None
            if self.cfg.max_boxes > 0:
                boxes, count = sc["boxes"][lo:hi].contiguous(), sc["box_count"][lo:hi].contiguous()
            self.batch.upload_worlds_at(envs, sc["grid"][lo:hi].contiguous(), boxes, count,
                                        sc["palette"][lo:hi].contiguous())
            obs = (torch.tensor(envs, device=self.device)[:, None] * A + torch.arange(A, device=self.device)).flatten()
            self.cams[obs] = sc["cams"][lo * A:hi * A]

    def _load_envs(self, envs):
        """Fresh worlds for the (sorted) env indices in `envs`, each in its current episode."""
        envs = [int(e) for e in envs]
        ep = self.episode.cpu()
        self._install(self._generate(envs, [int(ep[e]) for e in envs]))

    def _look_ahead(self):
        """Generate, in one go, the worlds of every env whose episode ends within the next _LOOKAHEAD
        steps (an env's clock and episode length say when), and file them by the step that needs them."""
        left = (self.episode_len - self.t).cpu()                # steps until each env finishes (>= 1)
        ep = self.episode.cpu()
        horizon = min(_LOOKAHEAD, int(self.episode_len.min()))  # no env finishes twice inside the window
        when = [(int(left[e]), e) for e in torch.nonzero(left <= horizon).flatten().tolist()]
        when.sort()
        envs = [e for _, e in when]
        chunks = self._generate(envs, [int(ep[e]) + 1 for e in envs])
        pos = 0
        for k in range(1, horizon + 1):
            n = sum(1 for w, _ in when if w == k)
            mine = envs[pos:pos + n]
            # the slices of the generated chunks that hold these envs
            parts, p = [], pos
            while p < pos + n:
                ci, off = divmod(p, _GEN_CHUNK)
                take = min(pos + n - p, _GEN_CHUNK - off)
                parts.append((chunks[ci], (off, off + take)))
                p += take
            self._ahead[self._step + k] = (mine, parts)
            pos += n

    def _render(self):
        if self.time_bar:
            rects = time_bar_rects(self.episode_len - self.t, self.episode_len, self.cfg.width, self.cfg.agents)
            self.batch.set_overlays(rects, self._bar_count)
        self.batch.render_batch(self.rgb, self.depth)
        return self.rgb, self.depth

    def reset(self):
        """Only needed once, right after construction."""
        self._load_envs(range(self.cfg.num_envs))
        self.batch.set_cameras(self.cams)
        self._started = True
        return self._render()

    def step(self, moves: torch.Tensor):
        """moves: CUDA float32 [num_obs][4] = (forward, strafe, dyaw, dpitch).  Returns
        (rgb [O][H][W][3] uint8, depth [O][H][W] float32, done [E] bool on the GPU); for a finished env
        the frames already show the first view of its next episode."""
        assert self._started, "call reset() once before step()"
        self.batch.move_agents(self.cams, moves.contiguous())
        if not self._ahead:
            self._look_ahead()
        self._step += 1
        self.t += 1
        done = self.t >= self.episode_len
        finished = torch.nonzero(done).flatten().cpu().tolist()       # the one device->host read of a step
        planned = self._ahead.pop(self._step, None)
        if finished:
            self.episode[done] += 1
            self.t[done] = 0
            if planned is not None and planned[0] == finished:
                for chunk, pick in planned[1]:
                    self._install([chunk], pick)
            else:
                self._load_envs(finished)
            self.batch.set_cameras(self.cams)
        rgb, depth = self._render()
        return rgb, depth, done

    def close(self):
        self.batch.destroy()
