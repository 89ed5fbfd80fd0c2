/*
 * laser_test_hooks.h -- controls of liblaser.so that exist for its tests only.
 *
 * Nothing here is part of the routing interface (the paper has no counterpart for either
 * call), and no result of a routing call depends on them except where stated.  Both settings
 * are process-wide, read when a routing call is enqueued, and not thread-safe: set them from
 * the thread that makes the calls, and restore them afterwards.
 */
#ifndef LASER_TEST_HOOKS_H_
#define LASER_TEST_HOOKS_H_

#ifdef __cplusplus
extern "C" {
#endif

enum {
  LASER_TEST_ROUTER_AUTO = 0,
  LASER_TEST_ROUTER_TILE = 1,          /* the 128-token-tile routers */
  LASER_TEST_ROUTER_SPLITK = 2,        /* the 16-token split-K router */
  LASER_TEST_ROUTER_TILE_ONESHOT = 3   /* as TILE, but every E > 32 takes the one-tile-per-block
                                          form of the tensor-memory router, not the persistent one */
};

/*
 * Overrides the choice between the 128-token-tile routers and the 16-token split-K router,
 * which is otherwise made from the number of tokens, so that small test shapes can run through
 * both.  It changes speed, never decisions (logits may differ in the last bits, as between any
 * two summation orders).  Returns the previous mode, or -1 (and changes nothing) for a mode
 * that is none of those above.
 */
int laser_test_set_router(int mode);

/*
 * Makes a bounded device-side wait run out without faulting or hanging anything: in every
 * routing call enqueued from now on, router tile `tile` of every layer writes its records but
 * publishes no ready flag, and the ordered selection gives up waiting after `wait_cycles` SM
 * clock cycles instead of its usual two seconds.  Such a call sets LASER_DEV_TIMEOUT in its
 * status word, marks the layer aborted, skips the layer's remaining selection and dispatch,
 * and returns; its outputs are unspecified but every access stays in bounds.
 * tile < 0 restores normal operation (wait_cycles is then ignored).  Returns 0, or -1 if
 * wait_cycles < 1 with tile >= 0.
 */
int laser_test_withhold_tile(int tile, long long wait_cycles);

/*
 * Enqueues one empty kernel (one block of 32 threads that does nothing) on cuda_stream (a
 * cudaStream_t passed as void*), so that a benchmark can time the launch floor of this library's
 * kernels on the machine at hand.  Returns 0, or -1 if the launch failed.
 */
int laser_test_launch_empty(void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* LASER_TEST_HOOKS_H_ */
