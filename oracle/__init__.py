"""CPU oracle of the Mirror-SD verify step.  Test infrastructure only: nothing on the
product path imports this package."""
